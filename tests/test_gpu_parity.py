"""GPU parity: the CUDA library, called through its C ABI binding, against the CPU oracle on the same seeded inputs.

Bars: mask bits, accepted lengths, node and token ids bit-exact; attention within max-abs 2e-2 for bf16
tensors (fp32 accumulation) and 1e-4 for fp32 tensors.  Because the bf16 workloads have outputs of
magnitude ~1e-3, each of them is also run with unit-variance q/k/v under a relative bound, and a "needle"
input reads the mask out of the attention output directly."""
import dataclasses

import numpy as np
import pytest
import torch

from mcsd_inputs import (attention_inputs, gammas, parent_array, seq_lens, verify_inputs, verify_logit_inputs,
                         workload)
from oracle import mcsd_oracle as orc
from tests.helpers import condition_uniforms, oracle_attention_rows, to_np

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2
TOL_F32 = 1e-4


@pytest.fixture(scope="module")
def m():
    from paper_2409_10644_b200 import build
    build.build()
    import paper_2409_10644_b200 as pkg
    return pkg


def _random_bfs_parent(rng, N, n_roots):
    parent = [-1] * n_roots
    lo, hi = 0, n_roots
    while len(parent) < N:
        start = len(parent)
        n_new = min(int(rng.integers(1, 3 * (hi - lo) + 1)), N - start)
        parent.extend(int(x) for x in np.sort(rng.integers(lo, hi, size=n_new)))
        lo, hi = start, len(parent)
    return np.asarray(parent[:N], dtype=np.int32)


# ----------------------------------------------------------------------------------------------
# mask
# ----------------------------------------------------------------------------------------------

def _check_mask(m, parent):
    tm = m.mcsd_build_mask(parent)
    torch.cuda.synchronize()
    depth, ls = orc.tree_levels(parent)
    bits = orc.pack_bitsets(orc.dense_mask(parent))
    got = tm.anc.cpu().numpy().view(np.uint64)
    assert np.array_equal(got[:, :bits.shape[1]], bits)
    assert not got[:, bits.shape[1]:].any()
    assert np.array_equal(tm.depth.cpu().numpy(), depth)
    assert tm.n_levels == len(ls) - 1
    assert np.array_equal(tm.level_start.cpu().numpy()[:len(ls)], ls)
    assert np.array_equal(tm.level_start_host, ls)
    return tm


def test_mask_bits_for_all_workload_trees(m):
    for i in range(1, 6):
        w = workload(i)
        _check_mask(m, parent_array(w.n_roots, w.branching))
    _check_mask(m, parent_array(2, (4, 3, 1, 1)))
    _check_mask(m, parent_array(16, (1, 1, 1, 1)))


@pytest.mark.parametrize("N", [1, 2, 63, 64, 65, 128, 129, 191, 192])
def test_mask_bits_random_trees(m, N):
    rng = np.random.default_rng(N)
    tm = _check_mask(m, _random_bfs_parent(rng, N, int(rng.integers(1, min(N, 9) + 1))))
    assert tm.words == (N + 63) // 64


def test_sliced_mask_is_a_row_count(m):
    # Section 3.2: rows/columns [0, n_active) of the big mask are the mask of the truncated tree
    w = workload(3)
    parent = parent_array(w.n_roots, w.branching)
    tm = m.mcsd_build_mask(parent)
    big = tm.anc.cpu().numpy().view(np.uint64)
    for gamma in range(len(w.branching) + 1):
        nb = int(m.n_active_from_gamma(tm.level_start_host, [gamma])[0])
        small = m.mcsd_build_mask(parent_array(w.n_roots, w.branching[:gamma]), words=tm.words)
        assert np.array_equal(big[:nb], small.anc.cpu().numpy().view(np.uint64))


# ----------------------------------------------------------------------------------------------
# attention
# ----------------------------------------------------------------------------------------------

def _run_attention(m, w, inp, lens, n_act, parent, scale=None):
    tm = m.mcsd_build_mask(parent)
    dev = inp["q"].device
    lens_d = torch.from_numpy(np.asarray(lens, dtype=np.int32)).to(dev)
    na_d = None if n_act is None else torch.from_numpy(np.asarray(n_act, dtype=np.int32)).to(dev)
    B, H, N, D = inp["q"].shape
    code = m.MCSD_F32 if inp["q"].dtype == torch.float32 else m.MCSD_BF16
    ws = torch.zeros(m.mcsd_tree_attention_workspace_bytes(B, H, N, D, inp["k_cache"].shape[2], code),
                     dtype=torch.uint8, device=dev)
    out = torch.full_like(inp["q"], float("nan"))
    m.mcsd_tree_attention(inp["q"], inp["k_cache"], inp["v_cache"], inp["k_tree"], inp["v_tree"], lens_d, na_d, tm,
                          out=out, softmax_scale=scale, workspace=ws)
    assert m.mcsd_workspace_status(ws) == 0
    return out


def _compare_attention(out, ref_rows, n_act, N, tol_abs, rel=False):
    worst = 0.0
    for (b, h), ref in ref_rows.items():
        nb = N if n_act is None else int(n_act[b])
        got = to_np(out[b, h]).astype(np.float64)
        if nb > 0:
            err = np.abs(got[:nb] - ref[:nb])
            assert np.isfinite(got[:nb]).all()
            if rel:
                scale = np.abs(ref[:nb]).max()
                assert err.max() <= tol_abs * scale, (b, h, err.max(), scale)
                rms = np.sqrt((err ** 2).mean()) / np.sqrt((ref[:nb] ** 2).mean())
                assert rms <= 1e-2, (b, h, rms)
            else:
                assert err.max() <= tol_abs, (b, h, err.max())
            worst = max(worst, err.max())
        assert np.isnan(got[nb:]).all()          # rows beyond n_active are not written
    return worst


def _all_pairs(B, H):
    return [(b, h) for b in range(B) for h in range(H)]


def _full_attention_case(m, w, std=None, rel=False, lens=None, n_act="gamma", pairs=None, poison=False, layer=0):
    parent = parent_array(w.n_roots, w.branching)
    inp = attention_inputs(w, layer, "cuda", std=std)
    lens = seq_lens(w) if lens is None else np.asarray(lens, dtype=np.int32)
    if isinstance(n_act, str):
        _, ls = orc.tree_levels(parent)
        n_act = None if w.gamma is None else np.array([orc.n_active_for_gamma(parent, int(g)) for g in gammas(w)])
    if poison:                                   # cache rows past the prefix and tree rows past the active nodes may hold anything
        for b in range(w.B):
            inp["k_cache"][b, :, int(lens[b]):] = float("nan")
            inp["v_cache"][b, :, int(lens[b]):] = float("nan")
            if n_act is not None:
                inp["k_tree"][b, :, int(n_act[b]):] = float("nan")
                inp["v_tree"][b, :, int(n_act[b]):] = float("nan")
    scale = 1.0 / np.sqrt(w.D)
    out = _run_attention(m, w, inp, lens, n_act, parent, scale)
    pairs = _all_pairs(w.B, w.H) if pairs is None else pairs
    ref = oracle_attention_rows(inp, lens, n_act, parent, scale, pairs)
    tol = TOL_F32 if w.dtype == "f32" else TOL_BF16
    return _compare_attention(out, ref, n_act, len(parent), tol, rel=rel)


def test_attention_tiny_fp32(m):
    _full_attention_case(m, workload(1))


def test_attention_llama7b_b1(m):
    _full_attention_case(m, workload(2))
    _full_attention_case(m, workload(2), std=1.0, rel=True)


def test_attention_dynamic_slice_reduced(m):
    # several key tiles plus a ragged tail, per-sequence gamma slices of the 109-node tree
    w = dataclasses.replace(workload(3), B=3, H=4, prefix=(300, 300))
    _full_attention_case(m, w, poison=True)
    _full_attention_case(m, w, std=1.0, rel=True, poison=True)


def test_attention_target_init_reduced(m):
    # ragged prefixes, 8 roots, 160-node tree sliced per sequence
    w = dataclasses.replace(workload(5), B=4, H=3, prefix=(5, 700))
    _full_attention_case(m, w, poison=True)
    _full_attention_case(m, w, std=1.0, rel=True, poison=True)


def test_attention_edge_cases(m):
    w = dataclasses.replace(workload(2), B=4, H=2, prefix=(0, 260))
    parent = parent_array(w.n_roots, w.branching)
    N = len(parent)
    # empty prefix, one-token prefix, exact tile multiple, ragged; empty and one-node trees
    _full_attention_case(m, w, std=1.0, rel=True, lens=[0, 1, 256, 259], n_act=np.array([N, 5, 0, 1]), poison=True)
    # head_dim 64 in bf16 and head_dim 128 in fp32 take the CUDA-core kernel
    _full_attention_case(m, dataclasses.replace(w, D=64), std=1.0, rel=True, lens=[7, 130, 33, 260])
    w32 = dataclasses.replace(workload(1), D=128, B=2, prefix=(40, 90))
    _full_attention_case(m, w32, lens=[40, 90])
    # largest tree
    wmax = dataclasses.replace(w, n_roots=8, branching=(1, 2, 2, 1, 1, 1, 1), B=2, prefix=(150, 150))
    assert wmax.n_nodes == 192
    _full_attention_case(m, wmax, std=1.0, rel=True, n_act=None)


def test_attention_half_filled_tiles(m):
    # A tile with at most 64 rows in use is fetched as a 64-row box and the rest of its slot keeps older data: prefix
    # ends and active-node counts on both sides of that limit, after full tiles and as the only tile, with NaN in
    # every row that must not be read.  Several heads per sequence, so that slots are reused within a block.
    w = dataclasses.replace(workload(3), B=8, H=4, prefix=(1, 400))
    N = w.n_nodes
    lens = [64, 65, 128 + 63, 128 + 64, 256 + 65, 1, 127, 384]
    n_act = np.array([N, 64, 65, 1, 63, N, 32, 100], dtype=np.int32)
    _full_attention_case(m, w, std=1.0, rel=True, lens=lens, n_act=n_act, poison=True)
    _full_attention_case(m, w, lens=lens[::-1], n_act=n_act, poison=True)


def test_attention_query_split_changes_between_segments(m):
    # Many short sequences of the 192-node tree with a different number of active nodes each: consecutive work
    # items of a thread block then split their query columns between the two softmax groups differently, and one
    # group may be a segment ahead of the other.  Run several times: a race would not fail every time.
    w = dataclasses.replace(workload(2), n_roots=8, branching=(1, 2, 2, 1, 1, 1, 1), B=12, H=3, prefix=(5, 300))
    assert w.n_nodes == 192
    rng = np.random.default_rng(7)
    lens = rng.integers(5, 301, w.B).astype(np.int32)
    n_act = np.array([192, 64, 17, 130, 8, 100, 192, 33, 160, 72, 129, 1], dtype=np.int32)
    for _ in range(3):
        _full_attention_case(m, w, std=1.0, rel=True, lens=lens, n_act=n_act, poison=True)


@pytest.mark.parametrize("G,case", [(4, "stacked"), (2, "stacked"), (8, "stacked"), (3, "stacked"), (8, "stacked_small"),
                                    (4, "too_wide"), (2, "f32")])
def test_attention_grouped_queries(m, G, case):
    # query heads share key/value heads; the tensor-core kernel stacks the queries of 8, 4 or 2 heads of a group into
    # one work unit when that divides the group and fits the 160 query columns of one pass (N = 45: two heads per
    # unit = 90 queries whatever G is, since four would be 180; G = 3 or N = 109: one head per unit, the key/value
    # head still shared; N = 15, G = 8: all eight heads = 120 queries); fp32 takes the CUDA-core kernel
    if case == "stacked":
        w = dataclasses.replace(workload(2), B=3, H=2 * G, prefix=(40, 600))          # N = 45: 90 stacked queries
    elif case == "stacked_small":
        w = dataclasses.replace(workload(1), dtype="bf16", D=128, B=2, H=G, prefix=(5, 300))   # N = 15: 120 queries
    elif case == "too_wide":
        w = dataclasses.replace(workload(3), B=2, H=G, prefix=(100, 300))              # N = 109: nothing to stack
    else:
        w = dataclasses.replace(workload(1), B=2, H=2 * G, prefix=(20, 128))           # fp32: CUDA-core kernel
    Hkv = w.H // G
    parent = parent_array(w.n_roots, w.branching)
    N = len(parent)
    inp = attention_inputs(w, 0, "cuda", std=1.0)
    for k in ("k_cache", "v_cache", "k_tree", "v_tree"):
        inp[k] = inp[k][:, :Hkv].contiguous()
    rng = np.random.default_rng(60 + G)
    lens = rng.integers(w.prefix[0], w.prefix[1] + 1, w.B).astype(np.int32)
    n_act = np.array([N, max(1, N // 3), N - 1][: w.B], dtype=np.int32)
    for b in range(w.B):
        inp["k_cache"][b, :, int(lens[b]):] = float("nan")
        inp["v_cache"][b, :, int(lens[b]):] = float("nan")
    scale = 1.0 / np.sqrt(w.D)
    out = _run_attention(m, w, inp, lens, n_act, parent, scale)
    host = {k: to_np(v) for k, v in inp.items()}
    ref = orc.tree_attention_gqa(host["q"], host["k_cache"], host["v_cache"], host["k_tree"], host["v_tree"],
                                 lens, n_act, parent, scale)
    rows = {(b, h): ref[b, h] for b in range(w.B) for h in range(w.H)}
    tol = TOL_F32 if w.dtype == "f32" else TOL_BF16
    _compare_attention(out, rows, n_act, N, tol, rel=(w.dtype != "f32"))


def test_attention_needle_reads_out_the_mask(m):
    # tree keys share one large score and carry one-hot values, the prefix scores 0 and carries zeros:
    # out[n][j] = 1/(depth(n)+1) exactly where node n may see node j
    for idx in (2, 3):
        w = workload(idx)
        parent = parent_array(w.n_roots, w.branching)
        N = len(parent)
        B, H, D, L = 2, 2, 128, 333
        dev = "cuda"
        z = lambda *s: torch.zeros(s, dtype=torch.bfloat16, device=dev)
        q, kc, vc, kt, vt = z(B, H, N, D), z(B, H, L, D), z(B, H, L, D), z(B, H, N, D), z(B, H, N, D)
        q[..., 0] = 8.0
        kt[..., 0] = 8.0
        g = torch.Generator(device=dev).manual_seed(3)
        kc[..., 1:] = torch.randn((B, H, L, D - 1), generator=g, device=dev).to(torch.bfloat16)
        for j in range(min(N, D)):
            vt[:, :, j, j] = 1.0
        inp = {"q": q, "k_cache": kc, "v_cache": vc, "k_tree": kt, "v_tree": vt}
        lens = [L, 77]
        out = _run_attention(m, w, inp, lens, None, parent, scale=1.0)
        ref = oracle_attention_rows(inp, lens, None, parent, 1.0, _all_pairs(B, H))
        mask = orc.dense_mask(parent)
        depth, _ = orc.tree_levels(parent)
        for (b, h), r in ref.items():
            got = to_np(out[b, h]).astype(np.float64)
            assert np.abs(got - r).max() <= 4e-3
            expect = mask[:, :min(N, D)] / (depth[:, None] + 1.0)
            assert np.abs(got[:, :min(N, D)] - expect).max() <= 4e-3


@pytest.mark.parametrize("idx", [3, 4, 5, 6, 7])
def test_attention_full_size_sampled(m, idx):
    # the workload at its full size, in the launch configuration the benchmark times; the oracle
    # checks a seeded sample of (sequence, head) pairs, every row of each
    w = workload(idx)
    rng = np.random.default_rng(idx)
    pairs = sorted({(int(rng.integers(w.B)), int(rng.integers(w.H))) for _ in range(6)} | {(0, 0), (w.B - 1, w.H - 1)})
    _full_attention_case(m, w, pairs=pairs)
    _full_attention_case(m, w, std=1.0, rel=True, pairs=pairs)
    if w.n_layers > 1:
        # the long-context workload repeats the step over 32 layers with independent seeded caches: also the
        # middle and the last layer, on their own samples of (sequence, head) pairs
        for layer in (w.n_layers // 2 - 1, w.n_layers - 1):
            lp = sorted({(int(rng.integers(w.B)), int(rng.integers(w.H))) for _ in range(4)})
            _full_attention_case(m, w, pairs=lp, layer=layer)
    torch.cuda.empty_cache()


def test_attention_dynamic_slice_depth6_reading(m):
    # The dynamic-slice configuration is quoted as "depth 8, 76 nodes"; its widths give 108 draft nodes and 76 is the
    # count of the first six levels.  The other tests take the widths; this is the other reading: every sequence
    # verified with draft length 6, i.e. 77 of the 109 rows of the mask built once for depth 8.
    w = workload(3)
    parent = parent_array(w.n_roots, w.branching)
    assert orc.n_active_for_gamma(parent, 6) == 77
    n_act = np.full(w.B, 77, dtype=np.int32)
    rng = np.random.default_rng(36)
    pairs = sorted({(int(rng.integers(w.B)), int(rng.integers(w.H))) for _ in range(5)} | {(0, 0)})
    _full_attention_case(m, w, n_act=n_act, pairs=pairs)
    _full_attention_case(m, w, std=1.0, rel=True, n_act=n_act, pairs=pairs)
    _verify_case(m, w, gamma=np.full(w.B, 6, dtype=np.int32))
    torch.cuda.empty_cache()


@pytest.mark.parametrize("H,L,roots,branching", [(1, 20000, 1, (4, 2, 2, 1)), (2, 9000, 8, (1, 2, 2, 1, 1, 1))])
def test_attention_one_work_item_cut_into_many_pieces(m, H, L, roots, branching):
    # One or two (sequence, head) pairs with a long prefix: every thread block gets a few tiles of the same work
    # item, so the item is merged from about as many pieces as there are blocks (the most the split allows).
    w = dataclasses.replace(workload(2), B=1, H=H, prefix=(L, L), n_roots=roots, branching=branching)
    _full_attention_case(m, w, std=1.0, rel=True, lens=[L - 77], n_act=None, poison=True)
    _full_attention_case(m, w, lens=[L], n_act=None)
    torch.cuda.empty_cache()


# ----------------------------------------------------------------------------------------------
# accept / reject
# ----------------------------------------------------------------------------------------------

def _verify_case(m, w, parent=None, B=None, V=None, gamma="workload", R=0, tweak=None, step=0):
    parent = parent_array(w.n_roots, w.branching) if parent is None else parent
    vin = verify_inputs(w, step, "cuda", parent=parent, B=B, V=V)
    B = vin["p"].shape[0]
    if isinstance(gamma, str):
        gamma = None if w.gamma is None else gammas(dataclasses.replace(w, B=B), step)
    if tweak is not None:
        tweak(vin)
    host = {k: to_np(v) for k, v in vin.items()}
    ua, ub = condition_uniforms(host["p"], host["q"], host["tokens"], parent, gamma, host["u_accept"], host["u_bonus"])
    ref = orc.verify_tree(host["p"], host["q"], host["tokens"], parent, gamma, ua, ub, R=R)
    tm = m.mcsd_build_mask(parent)
    dev = vin["p"].device
    g_d = None if gamma is None else torch.from_numpy(np.asarray(gamma, dtype=np.int32)).to(dev)
    got = m.mcsd_verify_tree(vin["p"], vin["q"], vin["tokens"], tm, g_d, torch.from_numpy(ua).to(dev),
                             torch.from_numpy(ub).to(dev), R=R)
    torch.cuda.synchronize()
    for k in ("accept_len", "out_tokens", "out_nodes", "best_root"):
        assert np.array_equal(got[k].cpu().numpy(), ref[k]), k
    if R > 0:
        assert np.array_equal(got["next_roots"].cpu().numpy(), ref["next_roots"])
    return ref


def test_verify_tiny_fp32_workload(m):
    _verify_case(m, workload(1), R=4)


def test_verify_llama7b_b1(m):
    ref = _verify_case(m, workload(2), R=8)
    assert ref["accept_len"][0] >= 0


def test_verify_dynamic_slice(m):
    _verify_case(m, workload(3))
    _verify_case(m, workload(3), step=1, R=2)


def test_verify_long_context_batch(m):
    ref = _verify_case(m, workload(4))
    assert ref["accept_len"].max() > 0          # the workload does accept draft tokens


def test_verify_target_initialised_forest(m):
    ref = _verify_case(m, workload(5), R=8)
    assert len(set(ref["best_root"].tolist())) > 1
    torch.cuda.empty_cache()


def test_verify_edge_cases(m):
    w = workload(1)
    # vocabulary sizes that are not a multiple of four take the scalar-load path
    for V in (5, 13, 1001):
        _verify_case(m, w, B=3, V=V, R=3)
    # gamma = 0: nothing is tested, the new token comes from the root's own row
    ref = _verify_case(m, w, B=2, gamma=np.array([0, 2]))
    assert ref["accept_len"][0] == 0
    # one-node tree
    _verify_case(m, w, parent=np.array([-1], dtype=np.int32), B=2, R=2)
    # draft equal to target: every first candidate is accepted down to the leaves
    def same(vin):
        vin["q"].copy_(vin["p"])
    ref = _verify_case(m, w, B=2, tweak=same)
    assert list(ref["accept_len"]) == [3, 3]
    # draft mass on a token the target never emits: all rejected, residual equals the target row
    def disjoint(vin):
        vin["p"][:, :, 0] = 0.0
        vin["p"].div_(vin["p"].sum(-1, keepdim=True))
        vin["q"].zero_()
        vin["q"][:, :, 0] = 1.0
        vin["tokens"][:, 1:] = 0
    ref = _verify_case(m, w, B=2, tweak=disjoint)
    assert list(ref["accept_len"]) == [0, 0]
    # fork-shaped tree of Section 3.2 with 16 chains, and the static (2; 4,3,1,1) configuration of Section 4.1
    w5 = workload(5)
    _verify_case(m, w5, parent=parent_array(16, (1, 1, 1, 1)), B=4, V=2000, gamma=np.array([4, 1, 2, 0]))
    _verify_case(m, w5, parent=parent_array(2, (4, 3, 1, 1)), B=4, V=2000, gamma=None, R=2)


# ----------------------------------------------------------------------------------------------
# accept / reject from logits: temperature > 0 and greedy (temperature 0)
# ----------------------------------------------------------------------------------------------

def _verify_logits_case(m, w, T, dtype, parent=None, B=None, V=None, gamma="workload", R=0, tweak=None, step=0):
    parent = parent_array(w.n_roots, w.branching) if parent is None else parent
    vin = verify_logit_inputs(w, T, dtype, step, "cuda", parent=parent, B=B, V=V)
    B = vin["target_logits"].shape[0]
    if isinstance(gamma, str):
        gamma = None if w.gamma is None else gammas(dataclasses.replace(w, B=B), step)
    if tweak is not None:
        tweak(vin)
    host = {k: to_np(v) for k, v in vin.items()}
    zt, zd = host["target_logits"], host["draft_logits"]
    ua, ub = host["u_accept"].copy(), host["u_bonus"].copy()
    keys = ("accept_len", "out_tokens", "out_nodes", "best_root", "next_roots")
    parts = []
    for b in range(B):                                   # sequences are independent; one at a time bounds the fp64 memory
        g = None if gamma is None else gamma[b:b + 1]
        if T > 0:
            pb = orc.softmax_temperature(zt[b:b + 1], T)
            qb = orc.softmax_temperature(zd[b:b + 1], T)
            ua[b:b + 1], ub[b:b + 1] = condition_uniforms(pb, qb, host["tokens"][b:b + 1], parent, g, ua[b:b + 1],
                                                          ub[b:b + 1], seed=777 + b)
            del pb, qb
            parts.append(orc.verify_tree_logits(zt[b:b + 1], zd[b:b + 1], T, host["tokens"][b:b + 1], parent, g,
                                                ua[b:b + 1], ub[b:b + 1], R=R))
        else:
            parts.append(orc.verify_tree_greedy(zt[b:b + 1], host["tokens"][b:b + 1], parent, g, R=R))
    ref = {k: np.concatenate([p_[k] for p_ in parts], axis=0) for k in keys}
    tm = m.mcsd_build_mask(parent)
    dev = vin["target_logits"].device
    g_d = None if gamma is None else torch.from_numpy(np.asarray(gamma, dtype=np.int32)).to(dev)
    if T > 0:
        got = m.mcsd_verify_tree_logits(vin["target_logits"], vin["draft_logits"], T, vin["tokens"], tm, g_d,
                                        torch.from_numpy(ua).to(dev), torch.from_numpy(ub).to(dev), R=R)
    else:
        got = m.mcsd_verify_tree_logits(vin["target_logits"], None, 0.0, vin["tokens"], tm, g_d, None, None, R=R)
    torch.cuda.synchronize()
    for k in ("accept_len", "out_tokens", "out_nodes", "best_root"):
        assert np.array_equal(got[k].cpu().numpy(), ref[k]), k
    if R > 0:
        assert np.array_equal(got["next_roots"].cpu().numpy(), ref["next_roots"])
    return ref


@pytest.mark.parametrize("T", [0.7, 1.0])
def test_verify_logits_tiny_fp32_workload(m, T):
    _verify_logits_case(m, workload(1), T, torch.float32, R=4)
    _verify_logits_case(m, workload(1), T, torch.bfloat16, B=3, R=4, step=1)


def test_verify_logits_llama_shapes_bf16(m):
    ref = _verify_logits_case(m, workload(2), 0.7, torch.bfloat16, R=8)
    assert ref["accept_len"][0] >= 0
    ref = _verify_logits_case(m, workload(4), 0.7, torch.bfloat16)
    assert ref["accept_len"].max() > 0


def test_verify_logits_dynamic_slice_and_forest(m):
    _verify_logits_case(m, workload(3), 0.7, torch.float32, R=2)
    ref = _verify_logits_case(m, workload(5), 1.0, torch.bfloat16, B=8, R=8)
    assert len(set(ref["best_root"].tolist())) > 1
    torch.cuda.empty_cache()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_verify_greedy_workloads(m, dtype):
    _verify_logits_case(m, workload(1), 0.0, dtype, R=4)
    ref = _verify_logits_case(m, workload(4), 0.0, dtype, R=2)
    assert ref["accept_len"].max() > 0
    _verify_logits_case(m, workload(3), 0.0, dtype, step=1)
    _verify_logits_case(m, workload(5), 0.0, dtype, B=8, R=8)
    torch.cuda.empty_cache()


def test_verify_logits_edge_cases(m):
    w = workload(1)
    for T in (0.7, 0.0):
        for dtype in (torch.float32, torch.bfloat16):
            # vocabulary sizes that are not a multiple of the vector width take the scalar-load path
            for V in (5, 13, 1001):
                _verify_logits_case(m, w, T, dtype, B=3, V=V, R=3)
            ref = _verify_logits_case(m, w, T, dtype, B=2, gamma=np.array([0, 2]))
            assert ref["accept_len"][0] == 0
            _verify_logits_case(m, w, T, dtype, parent=np.array([-1], dtype=np.int32), B=2, R=2)
    # ids the models can never emit (logit -inf), in different places for target and draft
    def masked(vin):
        vin["target_logits"][:, :, 0:40] = float("-inf")
        vin["draft_logits"][:, :, 20:60] = float("-inf")
        vin["tokens"][:, 1:3] = 5                          # candidates the target can never emit
    ref = _verify_logits_case(m, w, 0.7, torch.float32, B=2, tweak=masked, R=3)
    assert ref["out_tokens"].max() >= 40
    # draft equal to target: every first candidate is accepted down to the leaves
    def same(vin):
        vin["draft_logits"].copy_(vin["target_logits"])
    ref = _verify_logits_case(m, w, 1.0, torch.float32, B=2, tweak=same)
    assert list(ref["accept_len"]) == [3, 3]
    # greedy with equal largest logits: the lowest id wins; of two siblings with that token the first is followed
    def ties(vin):
        z = vin["target_logits"]
        z.clamp_(max=2.0)
        z[:, :, 700] = 4.0
        z[:, :, 300] = 4.0
        vin["tokens"][:, 1] = 700
        vin["tokens"][:, 2] = 300
        vin["tokens"][:, 5] = 300
        vin["tokens"][:, 6] = 300
    ref = _verify_logits_case(m, w, 0.0, torch.float32, B=2, tweak=ties, R=3)
    assert list(ref["out_nodes"][0][:2]) == [2, 5] and list(ref["next_roots"][0][:2]) == [300, 700]
    # large logits and a high temperature stay finite
    def big(vin):
        vin["target_logits"].mul_(30.0)
        vin["draft_logits"].mul_(30.0)
    _verify_logits_case(m, w, 50.0, torch.float32, B=2, tweak=big, R=2)
    w5 = workload(5)
    _verify_logits_case(m, w5, 0.7, torch.bfloat16, parent=parent_array(16, (1, 1, 1, 1)), B=4, V=2000,
                        gamma=np.array([4, 1, 2, 0]))
    _verify_logits_case(m, w5, 0.7, torch.float32, parent=parent_array(2, (4, 3, 1, 1)), B=4, V=2000, gamma=None, R=2)
    _verify_logits_case(m, w5, 0.0, torch.bfloat16, parent=parent_array(2, (4, 3, 1, 1)), B=4, V=2000, gamma=None, R=2)


def test_verify_paper_shaped_workloads(m):
    # the static (2; 4,3,1,1) forest and the early-stopped fork W = 16, D = 5 of Section 4.1, all three verify modes
    for idx in (6, 7):
        w = workload(idx)
        ref = _verify_case(m, w, R=2)
        assert ref["accept_len"].max() > 0
        _verify_logits_case(m, w, 0.7, torch.bfloat16, R=2, step=1)
        _verify_logits_case(m, w, 0.0, torch.bfloat16, R=2, step=1)
        torch.cuda.empty_cache()


def _roots_margin_ok(dist, picks, us, margin=2e-5):
    """True if every draw's uniform keeps `margin` (relative to the remaining mass) from the CDF edges of its id.
    The kernel forms the running sums in fp32 per lane and fp64 across warps (relative error around 1e-6); after the
    heaviest ids have been drawn the remaining ones are too light for the 1e-4 used elsewhere."""
    rest = np.array(dist, dtype=np.float64, copy=True)
    for t, u in zip(picks, us):
        if t < 0:
            break
        cs = np.cumsum(rest)
        z = cs[-1]
        lo = cs[t - 1] if t > 0 else -np.inf
        if min(u * z - lo, cs[t] - u * z) / z < margin:
            return False
        rest[t] = 0.0
    return True


@pytest.mark.parametrize("idx,R", [(1, 4), (5, 8), (7, 3)])
def test_sample_roots_matches_oracle(m, idx, R):
    w = workload(idx)
    parent = parent_array(w.n_roots, w.branching)
    B = min(w.B, 8)
    dev = "cuda"
    gam = None if w.gamma is None else gammas(dataclasses.replace(w, B=B))
    tm = m.mcsd_build_mask(parent)
    g_d = None if gam is None else torch.from_numpy(gam).to(dev)
    rng = np.random.default_rng(50 + idx)
    for mode in ("prob", "logits"):
        if mode == "prob":
            vin = verify_inputs(w, 0, dev, parent=parent, B=B)
            host = {k: to_np(v) for k, v in vin.items()}
            ph, qh = host["p"], host["q"]
        else:
            vin = verify_logit_inputs(w, 0.7, torch.bfloat16, 0, dev, parent=parent, B=B)
            host = {k: to_np(v) for k, v in vin.items()}
            ph = np.concatenate([orc.softmax_temperature(host["target_logits"][b:b + 1], 0.7) for b in range(B)])
            qh = np.concatenate([orc.softmax_temperature(host["draft_logits"][b:b + 1], 0.7) for b in range(B)])
        ua, ub = condition_uniforms(ph, qh, host["tokens"], parent, gam, host["u_accept"], host["u_bonus"])
        ref_v = orc.verify_tree(ph, qh, host["tokens"], parent, gam, ua, ub)
        # uniforms for the roots, redrawn (seeded) until none sits on a CDF edge the oracle evaluates
        ur = rng.uniform(0.001, 0.999, (B, R)).astype(np.float32)
        for b in range(B):
            _, dist = orc.stop_distribution(ph, qh, host["tokens"], parent, None if gam is None else gam[b], ua, b, ref_v)
            for _ in range(400):
                picks = orc.sample_without_replacement(dist, ur[b])
                if _roots_margin_ok(dist, picks, ur[b]):
                    break
                ur[b] = rng.uniform(0.001, 0.999, R).astype(np.float32)
            else:
                raise RuntimeError("could not move the root uniforms away from the thresholds")
        ref = orc.sample_roots(ph, qh, host["tokens"], parent, gam, ua, ref_v, ur)
        ws = m.new_workspace(m.mcsd_verify_tree_workspace_bytes(B, len(parent), w.V), dev)
        ua_d, ub_d, ur_d = (torch.from_numpy(x).to(dev) for x in (ua, ub, ur))
        if mode == "prob":
            vout = m.mcsd_verify_tree(vin["p"], vin["q"], vin["tokens"], tm, g_d, ua_d, ub_d, workspace=ws)
            got = m.mcsd_sample_roots(vin["p"], vin["q"], vout, tm, ur_d, ws)
        else:
            vout = m.mcsd_verify_tree_logits(vin["target_logits"], vin["draft_logits"], 0.7, vin["tokens"], tm, g_d, ua_d,
                                             ub_d, workspace=ws)
            got = m.mcsd_sample_roots(vin["target_logits"], vin["draft_logits"], vout, tm, ur_d, ws, temperature=0.7)
        torch.cuda.synchronize()
        assert np.array_equal(vout["accept_len"].cpu().numpy(), ref_v["accept_len"])
        assert np.array_equal(got.cpu().numpy(), ref), mode
        for b in range(B):
            row = [t for t in ref[b] if t >= 0]
            assert len(set(row)) == len(row)
        del vin
        torch.cuda.empty_cache()


def test_sample_roots_runs_out_of_mass(m):
    # a target row with mass on three ids only: the fourth and fifth root are -1
    w = workload(1)
    parent = np.array([-1], dtype=np.int32)
    dev = "cuda"
    V = 50
    p = torch.zeros((2, 1, V), device=dev)
    p[:, 0, 7] = 0.5
    p[:, 0, 20] = 0.25
    p[:, 0, 41] = 0.25
    q = torch.full((2, 1, V), 1.0 / V, device=dev)
    tm = m.mcsd_build_mask(parent)
    tokens = torch.zeros((2, 1), dtype=torch.int32, device=dev)
    half = torch.full((2, 1), 0.5, device=dev)
    ws = m.new_workspace(m.mcsd_verify_tree_workspace_bytes(2, 1, V), dev)
    vout = m.mcsd_verify_tree(p, q, tokens, tm, None, half, half, workspace=ws)
    ur = torch.tensor([[0.9, 0.1, 0.5, 0.5, 0.5], [0.1, 0.9, 0.5, 0.5, 0.5]], device=dev)
    got = m.mcsd_sample_roots(p, q, vout, tm, ur, ws).cpu().numpy()
    ref = np.stack([orc.sample_without_replacement(to_np(p[b, 0]), to_np(ur[b])) for b in range(2)])
    assert np.array_equal(got, ref)
    assert list(got[0]) == [41, 7, 20, -1, -1] and list(got[1]) == [7, 41, 20, -1, -1]
    del w


# ----------------------------------------------------------------------------------------------
# KV-cache update after acceptance
# ----------------------------------------------------------------------------------------------

@pytest.mark.parametrize("idx,dtype_D", [(5, None), (3, None), (1, None)])
def test_commit_kv_matches_oracle(m, idx, dtype_D):
    w = dataclasses.replace(workload(idx), B=4, H=3, prefix=(30, 60), n_layers=3)
    parent = parent_array(w.n_roots, w.branching)
    N = len(parent)
    tm = m.mcsd_build_mask(parent)
    dev = "cuda"
    layers = [attention_inputs(w, l, dev) for l in range(w.n_layers)]
    lens = np.array([30, 41, 57, 60][: w.B], dtype=np.int32)          # the last two run out of cache rows
    # what was accepted comes from the oracle's own verification (uniforms kept clear of its thresholds), for both
    # sides: the library's commit gets the oracle's accept_len / out_nodes / best_root, not the library's
    vin = verify_inputs(w, 0, dev, parent=parent, V=500)
    gam_h = None if w.gamma is None else gammas(w)
    hvin = {k: to_np(v) for k, v in vin.items()}
    ua, ub = condition_uniforms(hvin["p"], hvin["q"], hvin["tokens"], parent, gam_h, hvin["u_accept"], hvin["u_bonus"])
    hv = orc.verify_tree(hvin["p"], hvin["q"], hvin["tokens"], parent, gam_h, ua, ub)
    vout = {k: torch.from_numpy(np.ascontiguousarray(hv[k]).astype(np.int32)).to(dev)
            for k in ("accept_len", "out_tokens", "out_nodes", "best_root")}
    host_layers = [{k: to_np(v).copy() for k, v in l.items()} for l in layers]
    lens_d = torch.from_numpy(lens).to(dev)
    kc = m.layer_pointer_table([l["k_cache"] for l in layers])
    vc = m.layer_pointer_table([l["v_cache"] for l in layers])
    kt = m.layer_pointer_table([l["k_tree"] for l in layers])
    vt = m.layer_pointer_table([l["v_tree"] for l in layers])
    m.mcsd_commit_kv(kc, vc, kt, vt, lens_d, vout, tm, w.B, w.H, w.D, w.L_max, w.torch_dtype)
    torch.cuda.synchronize()
    new_ref = None
    for l, hl in zip(layers, host_layers):
        new_ref = orc.commit_kv(hl["k_cache"], hl["v_cache"], hl["k_tree"], hl["v_tree"], lens, hv["accept_len"],
                                hv["out_nodes"], hv["best_root"])
        assert np.array_equal(to_np(l["k_cache"]), hl["k_cache"])         # copies: bit-exact
        assert np.array_equal(to_np(l["v_cache"]), hl["v_cache"])
    assert np.array_equal(lens_d.cpu().numpy(), new_ref)
    assert (new_ref > lens).any()


# ----------------------------------------------------------------------------------------------
# bounded device-side waits
# ----------------------------------------------------------------------------------------------

def test_a_wait_that_runs_out_ends_in_a_status_and_a_usable_context(m):
    """The kernels' wait routine, given a signal that never comes and a short limit: the block gives up and exits, the
    workspace reports MCSD_ERR_TIMEOUT, and the same context and (re-zeroed) workspace then run a normal launch."""
    w = dataclasses.replace(workload(2), B=2, H=2, prefix=(100, 300))
    parent = parent_array(w.n_roots, w.branching)
    N = len(parent)
    ws = m.new_workspace(m.mcsd_tree_attention_workspace_bytes(w.B, w.H, N, w.D, w.L_max, m.MCSD_BF16), "cuda")
    assert m.mcsd_workspace_status(ws) == 0
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    m.mcsd_selftest_bounded_wait(ws, microseconds=2000)
    stop.record()
    torch.cuda.synchronize()
    assert m.mcsd_workspace_status(ws) == -7                      # MCSD_ERR_TIMEOUT
    assert "wait" in m.mcsd_status_string(-7)
    hdr = ws[:8].view(torch.int32).cpu().numpy()
    assert int(hdr[1]) == 42                                      # the code of the wait that gave up, not the follower's
    assert 0.5 <= start.elapsed_time(stop) <= 50.0                # about the 2 ms asked for, not the kernels' 2 s
    ws.zero_()
    inp = attention_inputs(w, 0, "cuda", std=1.0)
    lens = np.array([100, 300], dtype=np.int32)
    tm = m.mcsd_build_mask(parent)
    out = torch.full_like(inp["q"], float("nan"))
    m.mcsd_tree_attention(inp["q"], inp["k_cache"], inp["v_cache"], inp["k_tree"], inp["v_tree"],
                          torch.from_numpy(lens).cuda(), None, tm, out=out, softmax_scale=1 / np.sqrt(w.D), workspace=ws)
    assert m.mcsd_workspace_status(ws) == 0
    ref = oracle_attention_rows(inp, lens, None, parent, 1 / np.sqrt(w.D), [(0, 0), (1, 1)])
    for (b, h), rr in ref.items():
        err = np.abs(to_np(out[b, h]).astype(np.float64) - rr).max()
        assert err <= TOL_BF16 * np.abs(rr).max()
