"""Pins for the CPU oracle: it is checked against what the paper prints and what the
mathematics fixes, never against itself and never against the CUDA path."""
import itertools
import os

import numpy as np
import pytest
import torch

from mcsd_inputs import fork_parent_array, parent_array
from oracle import mcsd_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_counts.txt")


def _golden():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            k, v = line.split("=")
            out[k.strip()] = [int(t) for t in v.split()]
    return out


# ----------------------------------------------------------------------------
# trees and masks
# ----------------------------------------------------------------------------

def test_mask_sides_printed_for_fig1():
    g = _golden()
    # width 3, depth 2: the draft-initialised tree holds only the 6 draft tokens,
    # the target-initialised one adds the 3 target tokens in front (Section 3.1)
    draft = fork_parent_array(3, 2)
    target = fork_parent_array(3, 3)
    assert orc.dense_mask(draft).shape[0] == g["fig1_draft_init_mask_side"][0]
    assert orc.dense_mask(target).shape[0] == g["fig1_target_init_mask_side"][0]


def test_sliced_mask_sides_printed_for_fig2():
    g = _golden()
    parent = fork_parent_array(3, 3)
    # stopping after draft iteration i keeps i levels: gamma = i - 1 levels below the first one
    sides = [orc.sliced_mask(parent, gamma).shape[0] for gamma in (0, 1, 2)]
    assert sides == g["fig2_slice_sides"]


def test_counts_printed_for_static_configurations():
    g = _golden()
    parent = parent_array(2, (4, 3, 1, 1))
    depth, level_start = orc.tree_levels(parent)
    n_leaves = sum(1 for n in range(len(parent)) if not np.any(parent == n))
    assert (len(parent) - 2) // 2 == g["cfg_2_4_3_1_1_draft_tokens_per_root"][0]
    assert n_leaves == g["cfg_2_4_3_1_1_candidate_sequences"][0]
    assert int(depth.max()) == g["cfg_2_4_3_1_1_gamma"][0]
    parent = parent_array(1, (4, 2, 2, 1))
    depth, level_start = orc.tree_levels(parent)
    assert list(np.diff(level_start)[1:]) == g["cfg_4_2_2_1_level_sizes"]
    assert len(parent) - 1 == 44


def test_fork_mask_grows_linearly_expansion_tree_exponentially():
    # Section 3.2: fork-shaped trees add `width` tokens per level, expansion trees multiply
    fork = [len(fork_parent_array(3, d)) for d in (1, 2, 3, 4)]
    assert list(np.diff(fork)) == [3, 3, 3]
    exp = [len(parent_array(1, (3,) * d)) for d in (1, 2, 3, 4)]
    assert list(np.diff(exp)) == [9, 27, 81]


def _random_bfs_parent(rng, N, n_roots):
    """Random level-ordered tree: parents non-decreasing, every level non-empty."""
    parent = [-1] * n_roots
    lo, hi = 0, n_roots          # current parent level [lo, hi)
    while len(parent) < N:
        start = len(parent)
        n_new = int(rng.integers(1, max(2, min(N - start, 3 * (hi - lo)) + 1)))
        n_new = min(n_new, N - start)
        ps = np.sort(rng.integers(lo, hi, size=n_new))
        parent.extend(int(x) for x in ps)
        lo, hi = start, len(parent)
    return np.asarray(parent[:N], dtype=np.int32)


@pytest.mark.parametrize("N", [1, 2, 15, 63, 64, 65, 128, 129, 192])
def test_mask_invariants_on_random_trees(N):
    rng = np.random.default_rng(N)
    parent = _random_bfs_parent(rng, N, n_roots=int(rng.integers(1, min(N, 8) + 1)))
    depth, level_start = orc.tree_levels(parent)
    m = orc.dense_mask(parent)
    assert np.all(np.diag(m))
    assert not np.any(np.triu(m, 1))                      # nothing attends to a later node
    assert np.array_equal(m.sum(1), depth + 1)            # one bit per level of the root path
    for n in range(N):
        expect = np.zeros(N, dtype=bool)
        expect[n] = True
        if parent[n] >= 0:
            expect |= m[parent[n]]
        assert np.array_equal(m[n], expect)               # row = parent's row plus itself
    bits = orc.pack_bitsets(m)
    assert bits.shape == (N, (N + 63) // 64)
    for n in range(N):
        unpacked = [(int(bits[n, j // 64]) >> (j % 64)) & 1 for j in range(N)]
        assert unpacked == [int(x) for x in m[n]]
    # level_start brackets each depth
    for l in range(len(level_start) - 1):
        assert np.all(depth[level_start[l]:level_start[l + 1]] == l)


def test_sliced_mask_equals_mask_rebuilt_for_truncated_tree():
    for n_roots, br in [(1, (4, 2, 2, 1)), (8, (1, 2, 2, 1, 1, 1)), (1, (4, 2, 2, 1, 1, 1, 1, 1)), (3, (1, 1))]:
        parent = parent_array(n_roots, br)
        for gamma in range(len(br) + 1):
            truncated = parent_array(n_roots, br[:gamma])
            assert np.array_equal(orc.sliced_mask(parent, gamma), orc.dense_mask(truncated))
            assert orc.n_active_for_gamma(parent, gamma) == len(truncated)


def test_tree_levels_rejects_bad_orders():
    with pytest.raises(ValueError):
        orc.tree_levels([-1, 1])            # parent not earlier
    with pytest.raises(ValueError):
        orc.tree_levels([-1, 0, 1, 0])      # depth goes back down
    with pytest.raises(ValueError):
        orc.tree_levels([-1, -1, 1, 0])     # children out of parent order
    with pytest.raises(ValueError):
        orc.tree_levels([0, -1])            # node 0 is not a root


# ----------------------------------------------------------------------------
# attention
# ----------------------------------------------------------------------------

def _rand_attn(rng, B, H, N, D, L):
    f = lambda *s: rng.standard_normal(s)
    return f(B, H, N, D), f(B, H, L, D), f(B, H, L, D), f(B, H, N, D), f(B, H, N, D)


def _sdpa_causal_last(q_seq, k_seq, v_seq, scale):
    """Library causal attention over an explicit sequence [T][D]; returns all rows."""
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a))[None, None]
    o = torch.nn.functional.scaled_dot_product_attention(t(q_seq), t(k_seq), t(v_seq), is_causal=True, scale=scale)
    return o[0, 0].numpy()


def test_single_chain_tree_is_ordinary_causal_attention():
    rng = np.random.default_rng(1)
    B, H, N, D, L = 2, 3, 6, 16, 11
    q, kc, vc, kt, vt = _rand_attn(rng, B, H, N, D, L)
    parent = parent_array(1, (1,) * (N - 1))
    scale = 0.37
    out = orc.tree_attention(q, kc, vc, kt, vt, [L] * B, None, parent, scale)
    for b in range(B):
        for h in range(H):
            k_seq = np.concatenate([kc[b, h], kt[b, h]])
            v_seq = np.concatenate([vc[b, h], vt[b, h]])
            q_seq = np.concatenate([np.zeros((L, D)), q[b, h]])
            ref = _sdpa_causal_last(q_seq, k_seq, v_seq, scale)[L:]
            np.testing.assert_allclose(out[b, h], ref, rtol=0, atol=1e-12)


def test_each_node_equals_causal_attention_over_its_own_root_path():
    rng = np.random.default_rng(2)
    parent = parent_array(2, (2, 3, 1))
    N = len(parent)
    B, H, D, L = 2, 2, 8, 9
    q, kc, vc, kt, vt = _rand_attn(rng, B, H, N, D, L)
    lens = [L, 5]
    scale = 1.0 / np.sqrt(D)
    out = orc.tree_attention(q, kc, vc, kt, vt, lens, None, parent, scale)
    for b in range(B):
        for h in range(H):
            for n in range(N):
                path = []
                a = n
                while a >= 0:
                    path.append(a)
                    a = parent[a]
                path = path[::-1]
                k_seq = np.concatenate([kc[b, h, :lens[b]], kt[b, h, path]])
                v_seq = np.concatenate([vc[b, h, :lens[b]], vt[b, h, path]])
                q_seq = np.zeros_like(k_seq)
                q_seq[-1] = q[b, h, n]
                ref = _sdpa_causal_last(q_seq, k_seq, v_seq, scale)[-1]
                np.testing.assert_allclose(out[b, h, n], ref, rtol=0, atol=1e-12)


def test_attention_invariants():
    rng = np.random.default_rng(3)
    parent = parent_array(1, (3, 2))
    N = len(parent)
    B, H, D, L = 1, 2, 8, 7
    q, kc, vc, kt, vt = _rand_attn(rng, B, H, N, D, L)
    scale = 0.5
    base = orc.tree_attention(q, kc, vc, kt, vt, [L], None, parent, scale)
    mask = orc.dense_mask(parent)
    # changing K/V of nodes that are not on a node's root path leaves that node's output alone
    for n in range(N):
        kt2, vt2 = kt.copy(), vt.copy()
        others = ~mask[n]
        kt2[0, :, others] = rng.standard_normal((others.sum(), H, D)) * 5
        vt2[0, :, others] = rng.standard_normal((others.sum(), H, D)) * 5
        out = orc.tree_attention(q, kc, vc, kt2, vt2, [L], None, parent, scale)
        np.testing.assert_allclose(out[0, :, n], base[0, :, n], rtol=0, atol=1e-13)
    # each output is a convex combination of the values it may see
    for n in range(N):
        for h in range(H):
            vals = np.concatenate([vc[0, h], vt[0, h, mask[n]]])
            assert np.all(base[0, h, n] <= vals.max(0) + 1e-12)
            assert np.all(base[0, h, n] >= vals.min(0) - 1e-12)
    # no prefix at all: a root sees only itself, so its output is its own value row
    out0 = orc.tree_attention(q, kc, vc, kt, vt, [0], None, parent, scale)
    np.testing.assert_allclose(out0[0, :, 0], vt[0, :, 0], rtol=0, atol=1e-13)
    # sliced tree: rows beyond n_active are not produced, the others do not change
    outs = orc.tree_attention(q, kc, vc, kt, vt, [L], [4], parent, scale)
    np.testing.assert_allclose(outs[0, :, :4], base[0, :, :4], rtol=0, atol=1e-13)
    assert np.all(np.isnan(outs[0, :, 4:]))


# ----------------------------------------------------------------------------
# accept / reject
# ----------------------------------------------------------------------------

def _rand_dist(rng, *shape):
    x = rng.random(shape) ** 2 + 1e-3
    return x / x.sum(-1, keepdims=True)


def _forced_run(p, q, tokens, parent, forced, u_bonus=0.5):
    """Run the oracle with accept uniforms forced to 0 (accept if possible) or 1 (reject)."""
    N = len(parent)
    ua = np.ones((1, N))
    for c, v in forced.items():
        ua[0, c] = v
    ub = np.full((1, N), u_bonus)
    trace = []
    res = orc.verify_tree(p, q, tokens, parent, None, ua, ub, trace=trace)
    return res, trace


def _inverse_cdf_measure(dist, n_grid=200001):
    """Lebesgue measure of {u : inverse_cdf(dist, u) = t} estimated on a uniform grid."""
    us = (np.arange(n_grid) + 0.5) / n_grid
    counts = np.zeros(len(dist))
    for u in us:
        counts[orc.inverse_cdf(dist, u)] += 1
    return counts / n_grid


def test_inverse_cdf_samples_each_token_with_its_mass():
    rng = np.random.default_rng(4)
    dist = _rand_dist(rng, 7)
    dist[2] = 0.0
    dist = dist / dist.sum() * 3.0          # unnormalised input is allowed
    meas = _inverse_cdf_measure(dist, 20001)
    np.testing.assert_allclose(meas, dist / dist.sum(), atol=1e-4)
    assert orc.inverse_cdf(dist, 0.0) == 0
    assert orc.inverse_cdf(np.array([0.0, 0.0, 1.0, 0.0]), 0.3) == 2      # zero-mass ids are never drawn
    assert orc.inverse_cdf(np.array([0.5, 0.5]), 0.5) == 1                # strict comparison at an edge


@pytest.mark.parametrize("V,k", [(3, 1), (3, 2), (3, 3), (4, 1), (4, 2), (4, 3), (5, 1), (5, 2), (5, 3)])
def test_exact_enumeration_output_distribution_is_target(V, k):
    """One node with k sibling candidates drawn i.i.d. from q: the emitted token is distributed as p.

    k = 1 is plain speculative decoding (Section 2.1: the output distribution stays the target's)."""
    rng = np.random.default_rng(100 * V + k)
    p = _rand_dist(rng, 1, 1 + k, V)
    q = _rand_dist(rng, 1, 1 + k, V)
    if V == 4:
        q[0, 0, 1] = 0.0
        q[0, 0] /= q[0, 0].sum()          # a token the draft never proposes
        p[0, 0, 2] = 0.0
        p[0, 0] /= p[0, 0].sum()          # a token the target never emits
    parent = parent_array(1, (k,))
    emitted = np.zeros(V)
    for xs in itertools.product(range(V), repeat=k):
        w = np.prod([q[0, 0, x] for x in xs])
        if w == 0.0:
            continue
        tokens = np.array([[0] + list(xs)])
        # all-rejected run gives every stage's acceptance probability and the final residual
        res, trace = _forced_run(p, q, tokens, parent, {})
        a = [t["a"] for t in trace if "child" in t]
        stop = [t for t in trace if "stop" in t][0]
        assert len(a) == k and stop["stop"] == 0
        reach = 1.0
        for i in range(k):
            if a[i] > 0:
                forced = {1 + j: 1.0 for j in range(i)}
                forced[1 + i] = 0.0
                r2, _ = _forced_run(p, q, tokens, parent, forced)
                assert r2["accept_len"][0] == 1 and r2["out_tokens"][0, 0] == xs[i]
                assert r2["out_nodes"][0, 0] == 1 + i
            emitted[xs[i]] += w * reach * a[i]
            reach *= 1.0 - a[i]
        assert res["accept_len"][0] == 0
        emitted += w * reach * stop["dist"] / stop["dist"].sum()
    np.testing.assert_allclose(emitted, p[0, 0], rtol=0, atol=1e-12)


def test_two_level_tree_joint_distribution():
    """Tree (1; 2, 2): first emitted token ~ p(.), and given that it was an accepted
    candidate x1, the second emitted token ~ p(. | x1)."""
    V = 3
    rng = np.random.default_rng(7)
    p_root, q_root = _rand_dist(rng, V), _rand_dist(rng, V)
    P2, Q2 = _rand_dist(rng, V, V), _rand_dist(rng, V, V)      # conditional rows given the first token
    parent = parent_array(1, (2, 2))                            # nodes: 0 | 1 2 | 3 4 5 6
    first = np.zeros(V)
    joint = np.zeros((V, V))
    moved = np.zeros(V)
    for x1 in itertools.product(range(V), repeat=2):
        w1 = q_root[x1[0]] * q_root[x1[1]]
        for x2 in itertools.product(range(V), repeat=4):
            w = w1 * np.prod([Q2[x1[i // 2], x2[i]] for i in range(4)])
            tokens = np.array([[0, x1[0], x1[1], *x2]])
            p = np.zeros((1, 7, V))
            q = np.zeros((1, 7, V))
            p[0, 0], q[0, 0] = p_root, q_root
            for i in (0, 1):
                p[0, 1 + i], q[0, 1 + i] = P2[x1[i]], Q2[x1[i]]
            p[0, 3:] = 1.0 / V
            q[0, 3:] = 1.0 / V
            _, tr = _forced_run(p, q, tokens, parent, {})
            a1 = [t["a"] for t in tr if t.get("node") == 0]
            d1 = [t for t in tr if "stop" in t][0]["dist"]
            reach = 1.0
            for i in (0, 1):
                pr = reach * a1[i]
                reach *= 1.0 - a1[i]
                if pr == 0.0:
                    continue
                first[x1[i]] += w * pr
                moved[x1[i]] += w * pr
                c = 1 + i
                forced = {1 + j: 1.0 for j in range(i)}
                forced[c] = 0.0
                r2, tr2 = _forced_run(p, q, tokens, parent, forced)
                assert r2["out_nodes"][0, 0] == c
                a2 = [t["a"] for t in tr2 if t.get("node") == c]
                d2 = [t for t in tr2 if "stop" in t][0]
                assert d2["stop"] == c
                kids = [3 + 2 * i, 4 + 2 * i]
                reach2 = 1.0
                for j in (0, 1):
                    joint[x1[i], tokens[0, kids[j]]] += w * pr * reach2 * a2[j]
                    reach2 *= 1.0 - a2[j]
                joint[x1[i]] += w * pr * reach2 * d2["dist"] / d2["dist"].sum()
            first += w * reach * d1 / d1.sum()
    np.testing.assert_allclose(first, p_root, atol=1e-12)
    np.testing.assert_allclose(joint, moved[:, None] * P2, atol=1e-12)


def test_residual_matches_closed_form():
    """After m rejections the target-side distribution is max(p - s_m q, 0) / Z_m with
    s_0 = 0, Z_m = sum max(p - s_m q, 0), s_{m+1} = s_m + Z_m."""
    rng = np.random.default_rng(8)
    V, k = 50, 4
    p = _rand_dist(rng, 1, 1 + k, V)
    q = _rand_dist(rng, 1, 1 + k, V)
    parent = parent_array(1, (k,))
    tokens = np.array([[0] + [int(t) for t in rng.integers(0, V, k)]])
    s = 0.0
    for m in range(1, k + 1):
        par_m = parent_array(1, (m,))
        _, tr = _forced_run(p[:, :1 + m], q[:, :1 + m], tokens[:, :1 + m], par_m, {})
        dist = [t for t in tr if "stop" in t][0]["dist"]
        z = np.maximum(p[0, 0] - s * q[0, 0], 0).sum()
        s = s + z
        closed = np.maximum(p[0, 0] - s * q[0, 0], 0)
        np.testing.assert_allclose(dist, closed / closed.sum(), rtol=0, atol=1e-12)
        # acceptance probability of the next sibling against the closed form
        a = [t["a"] for t in tr if "child" in t]
        assert len(a) == m


def test_verify_special_cases():
    rng = np.random.default_rng(9)
    parent = parent_array(1, (2, 2, 1))
    N = len(parent)
    V = 11
    p = _rand_dist(rng, 2, N, V)
    tokens = rng.integers(0, V, (2, N)).astype(np.int32)
    ua = rng.random((2, N)) * 0.999
    ub = rng.random((2, N))
    # q = p: every first candidate is accepted, to full depth
    r = orc.verify_tree(p, p.copy(), tokens, parent, None, ua, ub)
    assert list(r["accept_len"]) == [3, 3]
    assert np.array_equal(r["out_nodes"][0, :3], [1, 3, 7])
    assert np.array_equal(r["out_tokens"][0, :3], tokens[0, [1, 3, 7]])
    # gamma slices the walk: with gamma = 1 only one level is tested, bonus from the raw row of the stop node
    r = orc.verify_tree(p, p.copy(), tokens, parent, [1, 0], ua, ub)
    assert list(r["accept_len"]) == [1, 0]
    assert r["out_tokens"][0, 1] == orc.inverse_cdf(p[0, 1], ub[0, 1])
    assert r["out_tokens"][1, 0] == orc.inverse_cdf(p[1, 0], ub[1, 0])
    assert np.all(r["out_tokens"][1, 1:] == -1) and np.all(r["out_nodes"][1] == -1)
    # draft puts all its mass on a token the target never emits: everything rejected,
    # the residual is the target row itself
    p2 = p.copy()
    p2[:, :, 0] = 0.0
    p2 /= p2.sum(-1, keepdims=True)
    q2 = np.zeros_like(p2)
    q2[:, :, 0] = 1.0
    tok0 = np.zeros_like(tokens)
    r = orc.verify_tree(p2, q2, tok0, parent, None, ua, ub)
    assert list(r["accept_len"]) == [0, 0]
    assert r["out_tokens"][0, 0] == orc.inverse_cdf(p2[0, 0], ub[0, 0])


def test_multi_root_selection_is_argmax_of_single_root_walks():
    rng = np.random.default_rng(10)
    n_roots, br = 4, (1, 2, 1)
    parent = parent_array(n_roots, br)
    N = len(parent)
    B, V = 6, 9
    p = _rand_dist(rng, B, N, V)
    q = _rand_dist(rng, B, N, V)
    tokens = rng.integers(0, V, (B, N)).astype(np.int32)
    ua, ub = rng.random((B, N)), rng.random((B, N))
    gam = rng.integers(0, 4, B)
    res = orc.verify_tree(p, q, tokens, parent, gam, ua, ub, R=3)
    mask = orc.dense_mask(parent)
    for b in range(B):
        lens = []
        for r in range(n_roots):
            # subtree of root r as a tree of its own
            nodes = [n for n in range(N) if mask[n, r]]
            remap = {n: i for i, n in enumerate(nodes)}
            sub_parent = np.array([-1 if parent[n] < 0 else remap[parent[n]] for n in nodes])
            rr = orc.verify_tree(p[b:b + 1, nodes], q[b:b + 1, nodes], tokens[b:b + 1, nodes], sub_parent,
                                 gam[b:b + 1], ua[b:b + 1, nodes], ub[b:b + 1, nodes], R=3)
            lens.append((int(rr["accept_len"][0]), rr, nodes))
        best = int(np.argmax([l[0] for l in lens]))        # first maximum = lowest root index
        assert res["best_root"][b] == best
        ln, rr, nodes = lens[best]
        assert res["accept_len"][b] == ln
        assert np.array_equal(res["out_nodes"][b, :ln], [nodes[i] for i in rr["out_nodes"][0, :ln]])
        # several roots: the selected root's own token is emitted first
        assert res["out_tokens"][b, 0] == tokens[b, best]
        assert np.array_equal(res["out_tokens"][b, 1:ln + 2], rr["out_tokens"][0, :ln + 1])
        assert np.array_equal(res["next_roots"][b], rr["next_roots"][0])


def test_next_roots_are_top_ids_with_ties_to_smaller_id():
    parent = parent_array(1, ())
    p = np.array([[[0.1, 0.3, 0.3, 0.2, 0.1]]])
    r = orc.verify_tree(p, p, np.zeros((1, 1), int), parent, None, np.zeros((1, 1)), np.full((1, 1), 0.5), R=4)
    assert list(r["next_roots"][0]) == [1, 2, 3, 0]
    assert r["out_tokens"][0, 0] == 2 and r["accept_len"][0] == 0


def test_acceptance_rate_definition():
    # Section 1: alpha = longest accepted draft length / maximum draft length
    parent = parent_array(1, (1, 1, 1, 1))
    rng = np.random.default_rng(11)
    p = _rand_dist(rng, 1, 5, 6)
    tokens = rng.integers(0, 6, (1, 5))
    r = orc.verify_tree(p, p.copy(), tokens, parent, None, np.full((1, 5), 0.5), np.full((1, 5), 0.5))
    assert r["accept_len"][0] / 4 == 1.0


def test_decision_margins_flag_uniforms_on_a_threshold():
    rng = np.random.default_rng(12)
    parent = parent_array(1, (2,))
    V = 5
    p = _rand_dist(rng, 1, 3, V)
    q = _rand_dist(rng, 1, 3, V)
    tokens = np.array([[0, 1, 2]])
    ratio = p[0, 0, 1] / q[0, 0, 1]
    ua = np.array([[0.5, min(ratio, 0.99), 0.5]])
    ub = np.full((1, 3), 0.5)
    m_acc, m_bon = orc.decision_margins(p, q, tokens, parent, None, ua, ub)
    if ratio < 0.99:
        assert m_acc[0, 1] < 1e-12
    assert np.isinf(m_acc[0, 0])
    # leaves can be stop nodes: their bonus margin is finite
    assert np.isfinite(m_bon[0, 1]) and np.isfinite(m_bon[0, 2])


def test_commit_kv_turns_the_accepted_path_into_ordinary_prefix():
    """Fig. 1 step 6: after the cache update the accepted tokens are plain prefix tokens, so causal attention of the
    deepest accepted token over the updated cache equals its tree-attention output before the update."""
    rng = np.random.default_rng(21)
    parent = parent_array(2, (2, 2, 1))
    N = len(parent)
    B, H, D, L_max = 3, 2, 8, 20
    q, kc, vc, kt, vt = _rand_attn(rng, B, H, N, D, L_max)
    lens = np.array([5, 11, 18], dtype=np.int32)            # the last sequence runs out of cache rows
    scale = 0.4
    before = orc.tree_attention(q, kc, vc, kt, vt, lens, None, parent, scale)
    mask = orc.dense_mask(parent)
    leaves = [n for n in range(N) if not np.any(parent == n)]
    best_root, accept_len, out_nodes = [], [], np.full((B, 4), -1)
    for b in range(B):
        leaf = leaves[int(rng.integers(len(leaves)))]
        path = [n for n in range(N) if mask[leaf, n]]
        cut = int(rng.integers(1, len(path) + 1))           # accept a prefix of the root path
        best_root.append(path[0]); accept_len.append(cut - 1); out_nodes[b, :cut - 1] = path[1:cut]
    kc2, vc2 = kc.copy(), vc.copy()
    new_lens = orc.commit_kv(kc2, vc2, kt, vt, lens, accept_len, out_nodes, best_root)
    for b in range(B):
        cnt = 1 + accept_len[b]
        assert new_lens[b] == min(L_max, lens[b] + cnt)
        assert np.array_equal(kc2[b, :, :lens[b]], kc[b, :, :lens[b]])          # old prefix untouched
        if lens[b] + cnt > L_max:
            continue
        last = best_root[b] if accept_len[b] == 0 else out_nodes[b, accept_len[b] - 1]
        for h in range(H):
            T = new_lens[b]
            q_seq = np.zeros((T, D)); q_seq[-1] = q[b, h, last]
            ref = _sdpa_causal_last(q_seq, kc2[b, h, :T], vc2[b, h, :T], scale)[-1]
            np.testing.assert_allclose(ref, before[b, h, last], rtol=0, atol=1e-12)
    # rows past the updated length keep their old content
    b = 0
    assert np.array_equal(kc2[b, :, new_lens[b]:], kc[b, :, new_lens[b]:])


# ----------------------------------------------------------------------------
# verification from logits: temperature and greedy (Fig. 1 step 4, Section 4.1)
# ----------------------------------------------------------------------------

def test_softmax_temperature_against_library_and_identities():
    import scipy.special
    rng = np.random.default_rng(20)
    z = rng.normal(0, 3, (2, 3, 17))
    for T in (1.0, 0.7, 2.5):
        s = orc.softmax_temperature(z, T)
        np.testing.assert_allclose(s, scipy.special.softmax(z / T, axis=-1), rtol=1e-13, atol=0)
        np.testing.assert_allclose(s.sum(-1), 1.0, rtol=1e-14)
        # adding a constant to a row changes nothing; log-ratios are logit differences over T
        np.testing.assert_allclose(orc.softmax_temperature(z + 123.0, T), s, rtol=1e-12)
        np.testing.assert_allclose(np.log(s[..., 3] / s[..., 5]), (z[..., 3] - z[..., 5]) / T, rtol=1e-11)
    # temperature T is the T = 1 distribution raised to 1/T and renormalised
    s1 = orc.softmax_temperature(z, 1.0)
    pw = s1 ** (1.0 / 0.7)
    np.testing.assert_allclose(orc.softmax_temperature(z, 0.7), pw / pw.sum(-1, keepdims=True), rtol=1e-12)
    # large logits must not overflow
    big = np.array([[1000.0, 999.0, -1000.0]])
    np.testing.assert_allclose(orc.softmax_temperature(big, 1.0)[0, :2], [1 / (1 + np.exp(-1)), 1 / (1 + np.exp(1))], rtol=1e-13)
    with pytest.raises(ValueError):
        orc.softmax_temperature(z, 0.0)


@pytest.mark.parametrize("T", [0.7, 1.0])
def test_exact_enumeration_output_distribution_is_tempered_target(T):
    """One node, two sibling candidates drawn i.i.d. from softmax(draft / T): the emitted token is distributed as
    softmax(target / T), written here with the library routine, not the oracle's own softmax."""
    import scipy.special
    V, k = 4, 2
    rng = np.random.default_rng(21)
    zt = rng.normal(0, 2, (1, 1 + k, V))
    zd = zt + rng.normal(0, 1.5, (1, 1 + k, V))
    q0 = scipy.special.softmax(zd[0, 0] / T)
    parent = parent_array(1, (k,))
    emitted = np.zeros(V)
    for xs in itertools.product(range(V), repeat=k):
        w = np.prod([q0[x] for x in xs])
        tokens = np.array([[0] + list(xs)])
        # acceptance probabilities of the two stages, from an all-rejected traced run
        trace = []
        ua = np.full((1, 1 + k), 1.0)
        ub = np.full((1, 1 + k), 0.5)
        orc.verify_tree_logits(zt, zd, T, tokens, parent, None, ua, ub, trace=trace)
        a = [t["a"] for t in trace if "child" in t]
        stop = [t for t in trace if "stop" in t][0]
        reach = 1.0
        for i in range(k):
            emitted[xs[i]] += w * reach * a[i]
            reach *= 1.0 - a[i]
        emitted += w * reach * stop["dist"] / stop["dist"].sum()
    np.testing.assert_allclose(emitted, scipy.special.softmax(zt[0, 0] / T), rtol=0, atol=1e-12)


def _toy_model_logits(seq, V):
    """A deterministic toy 'target model': next-token logits as a function of the whole token sequence."""
    rng = np.random.default_rng(abs(hash(tuple(int(t) for t in seq))) % (2 ** 32))
    return rng.normal(0, 1, V)


def _toy_tree(parent, V, prefix, seed, hit_rate):
    """Tokens for every node (a child repeats the model's argmax with probability hit_rate) and, for every
    node, the toy model's logits after prefix + the node's root path."""
    rng = np.random.default_rng(seed)
    N = len(parent)
    tokens = np.zeros(N, dtype=np.int64)
    paths = [None] * N
    logits = np.zeros((N, V))
    for n in range(N):
        if parent[n] < 0:
            tokens[n] = rng.integers(0, V)
            paths[n] = list(prefix) + [tokens[n]]
        else:
            top = int(np.argmax(logits[parent[n]]))
            tokens[n] = top if rng.random() < hit_rate else rng.integers(0, V)
            paths[n] = paths[parent[n]] + [tokens[n]]
        logits[n] = _toy_model_logits(paths[n], V)
    return tokens, logits, paths


@pytest.mark.parametrize("n_roots,branching", [(1, (3, 2, 1)), (1, (1, 1, 1, 1)), (2, (2, 2, 1)), (3, (2, 1))])
def test_greedy_verification_reproduces_autoregressive_greedy_decoding(n_roots, branching):
    """Temperature 0: what verification emits after a root is exactly what the target would have produced
    token by token (speculative decoding does not change greedy output), and it stops at the first level where no
    candidate carries the target's argmax."""
    V = 7
    parent = parent_array(n_roots, branching)
    depth, level_start = orc.tree_levels(parent)
    hits = 0
    for seed in range(40):
        prefix = [seed % V, (3 * seed) % V]
        tokens, logits, paths = _toy_tree(parent, V, prefix, seed, 0.7)
        r = orc.verify_tree_greedy(logits[None], tokens[None], parent, None, R=2)
        ln = int(r["accept_len"][0])
        root = int(r["best_root"][0])
        emitted = [int(t) for t in r["out_tokens"][0] if t >= 0]
        assert len(emitted) == ln + 1 + (1 if n_roots > 1 else 0)
        # autoregressive greedy decode of the toy model from prefix + chosen root token
        seq = list(prefix) + [int(tokens[root])]
        want = [int(tokens[root])] if n_roots > 1 else []
        for _ in range(ln + 1):
            nxt = int(np.argmax(_toy_model_logits(seq, V)))
            want.append(nxt)
            seq.append(nxt)
        assert emitted == want
        # accepted nodes form a root path of the chosen root
        u = root
        for i in range(ln):
            c = int(r["out_nodes"][0, i])
            assert parent[c] == u and tokens[c] == emitted[i + (1 if n_roots > 1 else 0)]
            u = c
        # the walk could not have gone further: no child of the stop node carries its argmax (or the tree ends)
        kids = [c for c in range(len(parent)) if parent[c] == u]
        assert all(tokens[c] != emitted[-1] for c in kids)
        # no other root gets further (brute force over all root paths)
        for n in range(len(parent)):
            path = []
            v = n
            while v >= 0:
                path.append(v)
                v = parent[v]
            path = path[::-1]
            # siblings are tried in order, so of several siblings with the argmax token the first is followed
            def first_hit(par):
                top = int(np.argmax(logits[par]))
                hit = [c for c in range(len(parent)) if parent[c] == par and tokens[c] == top]
                return hit[0] if hit else -1
            ok = all(path[i + 1] == first_hit(path[i]) for i in range(len(path) - 1))
            if ok:
                assert len(path) - 1 <= ln
                if len(path) - 1 == ln:
                    assert path[0] >= root
        assert list(r["next_roots"][0]) == list(np.argsort(-logits[u], kind="stable")[:2])
        hits += ln
    assert hits > 0                                     # the cases do accept something


def test_greedy_is_the_low_temperature_limit_and_honours_gamma_and_ties():
    rng = np.random.default_rng(23)
    V = 9
    parent = parent_array(2, (2, 2, 1))
    N = len(parent)
    for trial in range(20):
        zt = rng.normal(0, 1, (3, N, V))
        zt[np.arange(3)[:, None], np.arange(N)[None, :], rng.integers(0, V, (3, N))] += 2.0   # a clear winner
        zd = zt + rng.normal(0, 0.5, (3, N, V))
        # a cold draft only ever proposes its own most likely token; some of those agree with the target
        tokens = rng.integers(0, V, (3, N))
        for c in range(N):
            if parent[c] >= 0:
                src = zt if rng.random() < 0.6 else zd
                tokens[:, c] = np.argmax(src[:, parent[c]], axis=-1)
        gamma = rng.integers(0, 4, 3)
        ua = rng.uniform(0.01, 0.99, (3, N))
        ub = rng.uniform(0.01, 0.99, (3, N))
        cold = orc.verify_tree_logits(zt, zd, 1e-3, tokens, parent, gamma, ua, ub, R=1)
        greedy = orc.verify_tree_greedy(zt, tokens, parent, gamma, R=1)
        for key in ("accept_len", "out_tokens", "out_nodes", "best_root", "next_roots"):
            assert np.array_equal(cold[key], greedy[key]), key
        assert np.all(greedy["accept_len"] <= gamma)
    # equal largest logits: the lowest id wins, for acceptance and for the new token
    z = np.zeros((1, 3, 4))
    z[0, 0] = [1.0, 5.0, 5.0, 0.0]
    z[0, 1] = [2.0, 2.0, 2.0, 2.0]
    r = orc.verify_tree_greedy(z, np.array([[0, 2, 1]]), parent_array(1, (2,)), None, R=3)
    assert r["accept_len"][0] == 1 and r["out_nodes"][0, 0] == 2
    assert list(r["out_tokens"][0]) == [1, 0, -1] and list(r["next_roots"][0]) == [0, 1, 2]
    assert orc.argmax_lowest([3.0, 7.0, 7.0]) == 1


# ----------------------------------------------------------------------------
# several target-side tokens for the next tree (Section 3.1)
# ----------------------------------------------------------------------------

def test_sampling_without_replacement_follows_the_sequential_law():
    """Pairs (t1, t2) drawn with a fine grid of uniforms occur with frequency P(t1) * P(t2) / (1 - P(t1)), the law of
    sequential sampling without replacement, written out here independently of the oracle's own routine."""
    dist = np.array([0.5, 0.0, 1.5, 1.0, 2.0])            # unnormalised, one id without mass
    P = dist / dist.sum()
    G = 160
    grid = (np.arange(G) + 0.5) / G
    counts = np.zeros((5, 5))
    for u1 in grid:
        for u2 in grid:
            t = orc.sample_without_replacement(dist, [u1, u2])
            assert t[0] != t[1]
            counts[t[0], t[1]] += 1
    freq = counts / G ** 2
    want = np.zeros((5, 5))
    for a in range(5):
        for b in range(5):
            if a != b and P[a] > 0 and P[b] > 0:
                want[a, b] = P[a] * P[b] / (1.0 - P[a])
    assert np.abs(freq - want).max() < 2.5 / G
    assert counts[1].sum() == 0 and counts[:, 1].sum() == 0


def test_sampling_without_replacement_special_cases():
    dist = np.array([0.2, 0.3, 0.5])
    # all ids drawn: a permutation; with more draws than ids with mass, the rest is -1
    t = orc.sample_without_replacement(dist, [0.9, 0.1, 0.5, 0.5])
    assert sorted(t[:3]) == [0, 1, 2] and t[3] == -1
    assert list(t[:3]) == [2, 0, 1]                        # 0.9 -> id 2; then {0.2, 0.3}: 0.1 -> id 0; then id 1
    # in token-id order with a strict comparison: a uniform exactly on a CDF edge takes the next id
    assert orc.sample_without_replacement(np.array([1.0, 1.0]), [0.5])[0] == 1
    # point mass
    assert list(orc.sample_without_replacement(np.array([0.0, 3.0, 0.0]), [0.7, 0.7])) == [1, -1]


def test_sample_roots_draws_from_the_residual_of_the_stop_node():
    rng = np.random.default_rng(31)
    V = 6
    parent = parent_array(1, (2, 1))
    N = len(parent)
    p = _rand_dist(rng, 2, N, V)
    q = _rand_dist(rng, 2, N, V)
    tokens = rng.integers(0, V, (2, N))
    ua = np.ones((2, N))                                    # reject everything: stop at the root after two rejections
    ub = np.full((2, N), 0.5)
    v = orc.verify_tree(p, q, tokens, parent, None, ua, ub)
    assert list(v["accept_len"]) == [0, 0]
    ur = rng.uniform(0.05, 0.95, (2, 3))
    roots = orc.sample_roots(p, q, tokens, parent, None, ua, v, ur)
    for b in range(2):
        r1 = np.maximum(p[b, 0] - q[b, 0], 0.0); r1 /= r1.sum()          # residual after the first rejection
        r2 = np.maximum(r1 - q[b, 0], 0.0)                                # and after the second
        if r2.sum() > 0:
            r2 /= r2.sum()
        else:
            r2 = p[b, 0]
        stop, dist = orc.stop_distribution(p, q, tokens, parent, None, ua, b, v)
        assert stop == 0
        np.testing.assert_allclose(dist / dist.sum(), r2 / r2.sum(), atol=1e-12)
        n_pos = int((r2 > 0).sum())
        got = [int(t) for t in roots[b] if t >= 0]
        assert len(got) == min(3, n_pos) and len(set(got)) == len(got) and all(r2[t] > 0 for t in got)
        assert all(t == -1 for t in roots[b][len(got):])
    # an accepted path: the distribution is the target row of the deepest accepted node
    ua0 = np.zeros((2, N))
    v2 = orc.verify_tree(p, q, tokens, parent, None, ua0, ub)
    for b in range(2):
        stop, dist = orc.stop_distribution(p, q, tokens, parent, None, ua0, b, v2)
        assert stop == int(v2["out_nodes"][b, v2["accept_len"][b] - 1])
        np.testing.assert_allclose(dist, p[b, stop], atol=0)


def test_grouped_query_attention_is_attention_with_repeated_kv_heads():
    rng = np.random.default_rng(41)
    B, Hkv, G, D, L = 2, 2, 3, 8, 11
    parent = parent_array(1, (2, 2))
    N = len(parent)
    q = rng.normal(size=(B, Hkv * G, N, D))
    kc, vc = rng.normal(size=(B, Hkv, L, D)), rng.normal(size=(B, Hkv, L, D))
    kt, vt = rng.normal(size=(B, Hkv, N, D)), rng.normal(size=(B, Hkv, N, D))
    lens, nact = [11, 4], [N, 3]
    got = orc.tree_attention_gqa(q, kc, vc, kt, vt, lens, nact, parent, 0.3)
    rep = lambda x: np.repeat(x, G, axis=1)                 # head h reads key/value head h // G
    want = orc.tree_attention(q, rep(kc), rep(vc), rep(kt), rep(vt), lens, nact, parent, 0.3)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-14)
    # heads of one group differ only through their queries
    q2 = q.copy()
    q2[:, 1] = q2[:, 0]
    got2 = orc.tree_attention_gqa(q2, kc, vc, kt, vt, lens, nact, parent, 0.3)
    np.testing.assert_allclose(got2[:, 1], got2[:, 0], rtol=0, atol=0)
    with pytest.raises(ValueError):
        orc.tree_attention_gqa(q[:, :5], kc, vc, kt, vt, lens, nact, parent, 0.3)


def test_grouped_query_attention_against_library_causal_attention_on_root_paths():
    """A pin outside the oracle: query head h of a grouped-query target, at node n, equals ordinary causal attention
    (library routine) of that query over [prefix of key/value head h // G | the root path of n], last position."""
    rng = np.random.default_rng(43)
    B, Hkv, G, D = 2, 2, 3, 8
    parent = parent_array(2, (2, 1, 2))
    N = len(parent)
    lens = [9, 0]
    L = max(lens)
    q = rng.normal(size=(B, Hkv * G, N, D))
    kc, vc = rng.normal(size=(B, Hkv, L, D)), rng.normal(size=(B, Hkv, L, D))
    kt, vt = rng.normal(size=(B, Hkv, N, D)), rng.normal(size=(B, Hkv, N, D))
    scale = 0.41
    got = orc.tree_attention_gqa(q, kc, vc, kt, vt, lens, None, parent, scale)
    for b in range(B):
        for h in range(Hkv * G):
            hk = h // G
            for n in range(N):
                path = []
                u = n
                while u >= 0:
                    path.append(u)
                    u = int(parent[u])
                path = path[::-1]
                k_seq = np.concatenate([kc[b, hk, :lens[b]], kt[b, hk, path]])
                v_seq = np.concatenate([vc[b, hk, :lens[b]], vt[b, hk, path]])
                q_seq = np.zeros_like(k_seq)
                q_seq[-1] = q[b, h, n]
                ref = _sdpa_causal_last(q_seq, k_seq, v_seq, scale)[-1]
                np.testing.assert_allclose(got[b, h, n], ref, rtol=0, atol=1e-12)
    # a wrong head map must show: with the other key/value head the outputs differ
    swapped = orc.tree_attention_gqa(q, kc[:, ::-1], vc[:, ::-1], kt[:, ::-1], vt[:, ::-1], lens, None, parent, scale)
    assert np.abs(swapped - got).max() > 1e-3


def test_decision_margins_on_hand_written_rows():
    """Both halves of decision_margins against distances written out by hand.

    Root with two children over a vocabulary of three.  Root row: p = (0.5, 0.3, 0.2), q = (0.25, 0.25, 0.5).
    Child 1 carries token 0 (ratio p/q = 2, unclamped), child 2 carries token 2 (tested only after a rejection,
    against the residual max(p - q, 0) = (0.25, 0.05, 0) / 0.3: ratio 0 / 0.5 = 0)."""
    parent = parent_array(1, (2,))
    p = np.array([[[0.5, 0.3, 0.2], [0.2, 0.2, 0.6], [0.1, 0.7, 0.2]]])
    q = np.array([[[0.25, 0.25, 0.5], [0.3, 0.3, 0.4], [0.3, 0.3, 0.4]]])
    tokens = np.array([[9, 0, 2]])
    # (a) first child accepted (u = 0.75 < min(1, 2)): only its test is made; no new token at the root
    ua = np.array([[0.5, 0.75, 0.4]])
    ub = np.array([[0.5, 0.5, 0.95]])
    m_acc, m_bon = orc.decision_margins(p, q, tokens, parent, None, ua, ub)
    assert m_acc[0, 1] == pytest.approx(2.0 - 0.75, abs=1e-12)         # distance from the unclamped ratio
    assert np.isinf(m_acc[0, 0]) and np.isinf(m_acc[0, 2])             # root never tested; sibling 2 not reached
    assert np.isinf(m_bon[0, 0])
    # leaves stop with their own row p: cumulative sums (0.2, 0.4, 1.0) and (0.1, 0.8, 1.0)
    assert m_bon[0, 1] == pytest.approx(min(0.5 - 0.4, 1.0 - 0.5), abs=1e-12)      # u = 0.5 falls in token 2
    assert m_bon[0, 2] == pytest.approx(min(0.95 - 0.8, 1.0 - 0.95), abs=1e-12)    # u = 0.95 falls in token 2
    # (b) a uniform above 1 is not possible, so make the first test fail through the tokens: child 1 now carries
    # token 2 (ratio 0.2 / 0.5 = 0.4), child 2 token 0, tested against the residual (0.25, 0.05, 0) / 0.3:
    # ratio (0.25 / 0.3) / 0.25 = 10 / 3
    tokens_b = np.array([[9, 2, 0]])
    ua_b = np.array([[0.5, 0.9, 0.25]])
    m_acc, m_bon = orc.decision_margins(p, q, tokens_b, parent, None, ua_b, ub)
    assert m_acc[0, 1] == pytest.approx(0.9 - 0.4, abs=1e-12)
    assert m_acc[0, 2] == pytest.approx(10.0 / 3.0 - 0.25, abs=1e-12)
    assert np.isinf(m_bon[0, 0])                                       # second child accepted: no stop at the root
    # (c) both rejected: child 2 carries token 2 again, whose residual mass is 0 -> ratio 0, rejected for any u.
    # After it the residual is max((0.25, 0.05, 0) / 0.3 - q, 0) = (7/12, 0, 0) -> all mass on token 0: every
    # u_bonus falls in token 0, whose cell is [0, 1]; the first token has no lower edge to cross (u * Z cannot fall
    # below zero), so the distance is the one to the upper edge, 1 - u.
    tokens_c = np.array([[9, 2, 2]])
    ua_c = np.array([[0.5, 0.9, 0.3]])
    ub_c = np.array([[0.3, 0.5, 0.5]])
    m_acc, m_bon = orc.decision_margins(p, q, tokens_c, parent, None, ua_c, ub_c)
    assert m_acc[0, 1] == pytest.approx(0.5, abs=1e-12)
    assert m_acc[0, 2] == pytest.approx(0.3 - 0.0, abs=1e-12)
    assert m_bon[0, 0] == pytest.approx(1.0 - 0.3, abs=1e-12)
    # a stop distribution with two cells: one rejection only (gamma cuts nothing, root has a single tested child)
    parent1 = parent_array(1, (1,))
    m_acc, m_bon = orc.decision_margins(p[:, :2], q[:, :2], np.array([[9, 2]]), parent1, None,
                                        np.array([[0.5, 0.9]]), np.array([[0.9, 0.5]]))
    # residual after rejecting token 2: (0.25, 0.05, 0) / 0.3, cumulative (5/6, 1, 1); u = 0.9 falls in token 1
    assert m_acc[0, 1] == pytest.approx(0.5, abs=1e-12)
    assert m_bon[0, 0] == pytest.approx(min(0.9 - 5.0 / 6.0, 1.0 - 0.9), abs=1e-12)
    # gamma = 0: the root is the stop node with its own row, cumulative (0.5, 0.8, 1.0); u = 0.9 -> token 2
    m_acc, m_bon = orc.decision_margins(p, q, tokens, parent, np.array([0]), ua, np.array([[0.9, 0.5, 0.5]]))
    assert np.isinf(m_acc).all()
    assert m_bon[0, 0] == pytest.approx(min(0.9 - 0.8, 1.0 - 0.9), abs=1e-12)
    assert np.isinf(m_bon[0, 1]) and np.isinf(m_bon[0, 2])
