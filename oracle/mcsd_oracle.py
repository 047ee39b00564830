"""CPU oracle for one-pass verification of a candidate token tree (fp64, numpy).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
verification path computes.  It is used by the tests, by the smoke check and
by the benchmark's CPU-baseline leg; the product path never calls it and it
shares no code with the CUDA library.

What each function follows:

* ``tree_levels``, ``dense_mask``, ``pack_bitsets``, ``sliced_mask`` -- the
  topology-aware causal mask of Section 2.2 / Fig. 1 step 2 (a tree token may
  attend to itself and to the tokens on its own root path) and the dynamic
  sliced mask of Section 3.2 (build the mask for the deepest tree once, keep
  the upper-left square that covers the first gamma draft levels).
* ``tree_attention`` -- tree attention of Section 2.2: every tree token attends
  to the whole prefix plus the tree tokens its mask row allows.  The method
  reaches exactly softmax(scale * q k^T) v over that key set, so the oracle is
  that definition written out.
* ``sample_without_replacement``, ``sample_roots`` -- Section 3.1: several new
  tokens, not one, are sampled from the target side to start the next tree.
* ``softmax_temperature``, ``verify_tree_logits``, ``verify_tree_greedy`` --
  Fig. 1 step 4 (next-token logits become distributions) at the two sampling
  temperatures of Section 4.1: 0.7 (probabilistic) and 0 (greedy).
* ``verify_tree`` -- Fig. 1 steps 4-6: per-sibling acceptance with probability
  min(1, p/q) (the speculative-sampling rule the paper inherits, Section 2.1),
  on rejection the target distribution becomes norm(max(p - q, 0)) and the next
  sibling is tried; the longest accepted candidate sequence is selected
  (Fig. 1 step 5; for several target-initialised roots, Section 3.1) and one
  more token is sampled from the target-side distribution at the stop node
  (Fig. 1 step 6).  It is an algorithm, so the steps are taken in that order.

Readings where the paper is silent (each is also listed in the design notes):
siblings are i.i.d. draws from the same q row and q is not changed between
siblings; ties between roots go to the lowest root index; a zero residual mass
falls back to the un-residualised row; the inverse CDF runs in token-id order
with a strict comparison against u * sum(dist); a candidate with q(x) = 0 is
accepted iff the current target mass on it is positive.

Parity pins: every function here is pinned by tests/test_oracle_pins.py
(counts printed in the paper, brute force on explicit root paths, a library
causal-attention routine, exact enumeration of the output distribution,
closed-form residuals).  The one exception is the *distribution* of the
multi-root selection, which by Section 3.1 has no closed form: for it only the
decision (argmax of per-root lengths) is pinned -- "parity unpinned" for the
distribution itself.
"""
from __future__ import annotations

from typing import List, Optional

import numpy as np


# ----------------------------------------------------------------------------
# tree topology and mask (Section 2.2, Fig. 1 step 2; Section 3.2)
# ----------------------------------------------------------------------------

def tree_levels(parent):
    """depth[n] (roots are level 0) and level_start[l] = index of the first node of level l.

    Raises ValueError unless nodes are in level order: parent[n] < n, depth
    non-decreasing with n, and the children of one node contiguous.
    """
    parent = np.asarray(parent, dtype=np.int64)
    N = len(parent)
    if N < 1:
        raise ValueError("empty tree")
    depth = np.zeros(N, dtype=np.int64)
    for n in range(N):
        if parent[n] >= n or parent[n] < -1:
            raise ValueError("parent[%d] = %d is not an earlier node" % (n, parent[n]))
        d, a = 0, parent[n]
        while a >= 0:
            d += 1
            a = parent[a]
        depth[n] = d
    if depth[0] != 0:
        raise ValueError("node 0 must be a root")
    for n in range(1, N):
        if depth[n] < depth[n - 1]:
            raise ValueError("nodes are not in level order at %d" % n)
        if parent[n] < parent[n - 1]:
            raise ValueError("children of one node are not contiguous at %d" % n)
    n_levels = int(depth[-1]) + 1
    level_start = np.zeros(n_levels + 1, dtype=np.int64)
    for l in range(n_levels):
        level_start[l] = int(np.argmax(depth == l))
    level_start[n_levels] = N
    return depth.astype(np.int32), level_start.astype(np.int32)


def dense_mask(parent):
    """mask[n][j] = True iff tree token n may attend to tree token j: j is n or an ancestor of n."""
    parent = np.asarray(parent, dtype=np.int64)
    N = len(parent)
    m = np.zeros((N, N), dtype=bool)
    for n in range(N):
        a = n
        while a >= 0:
            m[n, a] = True
            a = parent[a]
    return m


def pack_bitsets(mask):
    """Row n of the mask as 64-bit words: bit (j % 64) of word (j // 64) is mask[n][j]."""
    N = mask.shape[0]
    words = (mask.shape[1] + 63) // 64
    out = np.zeros((N, words), dtype=np.uint64)
    for n in range(N):
        for j in range(mask.shape[1]):
            if mask[n, j]:
                out[n, j // 64] |= np.uint64(1) << np.uint64(j % 64)
    return out


def n_active_for_gamma(parent, gamma):
    """Number of tree tokens kept for draft length gamma: the root level plus gamma draft levels."""
    depth, _ = tree_levels(parent)
    return int(np.sum(depth <= gamma))


def sliced_mask(parent, gamma):
    """Dynamic sliced mask (Section 3.2): the upper-left square of the full mask covering levels 0..gamma."""
    n = n_active_for_gamma(parent, gamma)
    return dense_mask(parent)[:n, :n]


# ----------------------------------------------------------------------------
# tree attention (Section 2.2)
# ----------------------------------------------------------------------------

def tree_attention(q, k_cache, v_cache, k_tree, v_tree, seq_lens, n_active, parent, scale):
    """out[b][h][n] = sum_j softmax_j(scale * <q_n, k_j>) v_j over the prefix keys 0..L_b-1
    and the tree keys allowed by mask row n, for n < n_active[b].  Rows n >= n_active[b] are NaN.

    q, k_tree, v_tree: [B][H][N][D]; k_cache, v_cache: [B][H][L_max][D]; any float dtype, widened to fp64.
    """
    q = np.asarray(q, dtype=np.float64)
    k_cache = np.asarray(k_cache, dtype=np.float64)
    v_cache = np.asarray(v_cache, dtype=np.float64)
    k_tree = np.asarray(k_tree, dtype=np.float64)
    v_tree = np.asarray(v_tree, dtype=np.float64)
    B, H, N, D = q.shape
    mask = dense_mask(parent)
    out = np.full((B, H, N, D), np.nan, dtype=np.float64)
    for b in range(B):
        L = int(seq_lens[b])
        Nb = N if n_active is None else int(n_active[b])
        if Nb == 0:
            continue
        allowed = np.concatenate([np.ones((Nb, L), dtype=bool), mask[:Nb, :Nb]], axis=1)
        for h in range(H):
            keys = np.concatenate([k_cache[b, h, :L], k_tree[b, h, :Nb]], axis=0)
            vals = np.concatenate([v_cache[b, h, :L], v_tree[b, h, :Nb]], axis=0)
            s = scale * (q[b, h, :Nb] @ keys.T)
            s = np.where(allowed, s, -np.inf)
            s = s - s.max(axis=1, keepdims=True)
            e = np.exp(s)
            w = e / e.sum(axis=1, keepdims=True)
            out[b, h, :Nb] = w @ vals
    return out


def tree_attention_gqa(q, k_cache, v_cache, k_tree, v_tree, seq_lens, n_active, parent, scale):
    """Tree attention (Section 2.2) for a target whose query heads share key/value heads (grouped-query attention).

    q is [B][H_q][N][D], the key/value tensors have H_kv heads, H_q = G * H_kv, and query head h reads key/value
    head h // G; everything else is tree_attention.  The paper's targets are multi-head models (G = 1).
    """
    Hq, Hkv = q.shape[1], k_tree.shape[1]
    if Hq % Hkv:
        raise ValueError("the number of query heads must be a multiple of the number of key/value heads")
    G = Hq // Hkv
    out = np.zeros(q.shape, dtype=np.float64)
    for h in range(Hq):
        kv = h // G
        out[:, h:h + 1] = tree_attention(q[:, h:h + 1], k_cache[:, kv:kv + 1], v_cache[:, kv:kv + 1],
                                         k_tree[:, kv:kv + 1], v_tree[:, kv:kv + 1], seq_lens, n_active, parent, scale)
    return out


# ----------------------------------------------------------------------------
# multi-candidate accept / reject (Fig. 1 steps 4-6, Section 3.1)
# ----------------------------------------------------------------------------

def accept_probability(pt, qd, x):
    """min(1, pt(x)/qd(x)); a candidate the draft gave zero mass is accepted iff the target mass is positive."""
    if qd[x] > 0.0:
        return min(1.0, pt[x] / qd[x])
    return 1.0 if pt[x] > 0.0 else 0.0


def residual(pt, qd, p_row):
    """norm(max(pt - qd, 0)); if nothing is left, fall back to the un-residualised row."""
    r = np.maximum(pt - qd, 0.0)
    z = r.sum()
    if z > 0.0:
        return r / z
    return p_row.copy()


def inverse_cdf(dist, u):
    """Smallest token id t with cumsum(dist)[t] > u * sum(dist); the last id with positive mass if none."""
    cs = np.cumsum(dist)
    hit = np.nonzero(cs > u * cs[-1])[0]
    if len(hit):
        return int(hit[0])
    pos = np.nonzero(dist > 0.0)[0]
    return int(pos[-1]) if len(pos) else len(dist) - 1


def node_decision(p_row, q_row, child_tokens, child_uniforms, tests: Optional[list] = None):
    """Try the children of one node in order.

    Returns (index of the first accepted child or None, distribution a bonus
    token would be drawn from if the walk stops here because every child was
    rejected).  ``tests`` collects (child index, acceptance probability,
    unclamped ratio) for every test actually made.
    """
    p_row = np.asarray(p_row, dtype=np.float64)
    qd = np.asarray(q_row, dtype=np.float64)
    pt = p_row.copy()
    for i, (x, u) in enumerate(zip(child_tokens, child_uniforms)):
        a = accept_probability(pt, qd, int(x))
        if tests is not None:
            ratio = pt[int(x)] / qd[int(x)] if qd[int(x)] > 0.0 else (np.inf if pt[int(x)] > 0.0 else 0.0)
            tests.append((i, a, ratio))
        if float(u) < a:
            return i, None
        pt = residual(pt, qd, p_row)
    return None, pt


def _children(parent, u):
    return [c for c in range(len(parent)) if parent[c] == u]


def verify_tree(p, q, tokens, parent, gamma, u_accept, u_bonus, R=0, trace: Optional[list] = None):
    """Accept/reject walk over the token tree, longest-sequence selection, bonus token.

    p, q: [B][N][V]; tokens, u_accept, u_bonus: [B][N]; gamma: [B] or None (full depth).
    Returns dict of int32 arrays: accept_len[B], out_tokens[B][n_levels+1] (-1 padded),
    out_nodes[B][n_levels] (-1 padded), best_root[B], next_roots[B][R].

    out_tokens = [root token if the tree has several roots] + accepted tokens + [bonus token].
    """
    parent = np.asarray(parent, dtype=np.int64)
    depth, level_start = tree_levels(parent)
    n_levels = len(level_start) - 1
    N = len(parent)
    B = p.shape[0]
    roots = [n for n in range(N) if parent[n] < 0]
    n_roots = len(roots)
    accept_len = np.zeros(B, dtype=np.int32)
    out_tokens = np.full((B, n_levels + 1), -1, dtype=np.int32)
    out_nodes = np.full((B, n_levels), -1, dtype=np.int32)
    best_root = np.zeros(B, dtype=np.int32)
    next_roots = np.full((B, max(R, 0)), -1, dtype=np.int32)
    for b in range(B):
        g = n_levels - 1 if gamma is None else int(gamma[b])
        results = []
        for r in roots:
            u = r
            path: List[int] = []
            while True:
                kids = _children(parent, u)
                dist = np.asarray(p[b, u], dtype=np.float64)
                if depth[u] == g or not kids:
                    break
                tests = [] if trace is not None else None
                idx, res = node_decision(p[b, u], q[b, u], [tokens[b, c] for c in kids],
                                         [u_accept[b, c] for c in kids], tests)
                if trace is not None:
                    for (i, a, ratio) in tests:
                        trace.append({"b": b, "root": r, "node": u, "child": kids[i], "a": a, "ratio": ratio})
                if idx is None:
                    dist = res
                    break
                path.append(kids[idx])
                u = kids[idx]
            bonus = inverse_cdf(dist, float(u_bonus[b, u]))
            if trace is not None:
                trace.append({"b": b, "root": r, "stop": u, "dist": dist.copy(), "bonus": bonus})
            results.append((len(path), r, path, bonus, dist))
        best = results[0]
        for cand in results[1:]:
            if cand[0] > best[0]:
                best = cand
        ln, r, path, bonus, dist = best
        accept_len[b] = ln
        best_root[b] = r
        toks = ([int(tokens[b, r])] if n_roots > 1 else []) + [int(tokens[b, c]) for c in path] + [bonus]
        out_tokens[b, :len(toks)] = toks
        out_nodes[b, :ln] = path
        if R > 0:
            order = np.argsort(-dist, kind="stable")
            next_roots[b, :] = order[:R]
    return {"accept_len": accept_len, "out_tokens": out_tokens, "out_nodes": out_nodes,
            "best_root": best_root, "next_roots": next_roots}


def decision_margins(p, q, tokens, parent, gamma, u_accept, u_bonus):
    """Distance of every supplied uniform from the decision thresholds it can meet.

    For every active node, evaluated on its own (the outcome at a node does not
    depend on how a walk reached it): margin_accept[b][c] = |u_accept - ratio|
    for each child test the node makes (ratio unclamped), and
    margin_bonus[b][n] = distance of u_bonus * Z from the two CDF edges that
    bracket it, divided by Z, for the distribution a stop at n would sample.
    Entries that no decision reads are +inf.
    """
    parent = np.asarray(parent, dtype=np.int64)
    depth, level_start = tree_levels(parent)
    n_levels = len(level_start) - 1
    N = len(parent)
    B = p.shape[0]
    m_acc = np.full((B, N), np.inf)
    m_bon = np.full((B, N), np.inf)
    for b in range(B):
        g = n_levels - 1 if gamma is None else int(gamma[b])
        for u in range(N):
            if depth[u] > g:
                continue
            kids = _children(parent, u)
            dist = np.asarray(p[b, u], dtype=np.float64)
            if depth[u] < g and kids:
                tests: list = []
                idx, res = node_decision(p[b, u], q[b, u], [tokens[b, c] for c in kids],
                                         [u_accept[b, c] for c in kids], tests)
                for (i, a, ratio) in tests:
                    m_acc[b, kids[i]] = abs(float(u_accept[b, kids[i]]) - ratio)
                if idx is not None:
                    continue
                dist = res
            cs = np.cumsum(dist)
            z = cs[-1]
            t = inverse_cdf(dist, float(u_bonus[b, u]))
            target = float(u_bonus[b, u]) * z
            lo = cs[t - 1] if t > 0 else -np.inf
            m_bon[b, u] = min(target - lo, cs[t] - target) / z
    return m_acc, m_bon


# ----------------------------------------------------------------------------
# several new tokens from the target side (Section 3.1)
# ----------------------------------------------------------------------------

def sample_without_replacement(dist, uniforms):
    """R distinct token ids drawn one after the other from an unnormalised distribution.

    Section 3.1 samples several tokens, not one, from the target's distribution to start the next candidate
    tree.  Reading taken here (the paper does not say how): the tokens are distinct; draw i is an inverse-CDF draw
    in token-id order (uniform uniforms[i]) from the distribution restricted to the ids not drawn yet, which is the
    usual sequential sampling without replacement.  When no mass is left the remaining entries are -1.
    """
    rest = np.array(dist, dtype=np.float64, copy=True)
    out = np.full(len(uniforms), -1, dtype=np.int32)
    for i, u in enumerate(uniforms):
        if not rest.sum() > 0.0:
            break
        t = inverse_cdf(rest, float(u))
        out[i] = t
        rest[t] = 0.0
    return out


def stop_distribution(p, q, tokens, parent, gamma_b, u_accept, b, verify_out):
    """Unnormalised distribution the new token of sequence b is drawn from: the target row of the stop node of the
    winning path, residualised once per candidate rejected there (Fig. 1 steps 4-6)."""
    parent = np.asarray(parent, dtype=np.int64)
    depth, level_start = tree_levels(parent)
    n_levels = len(level_start) - 1
    g = n_levels - 1 if gamma_b is None else int(gamma_b)
    ln = int(verify_out["accept_len"][b])
    stop = int(verify_out["out_nodes"][b, ln - 1]) if ln > 0 else int(verify_out["best_root"][b])
    kids = _children(parent, stop)
    dist = np.asarray(p[b, stop], dtype=np.float64)
    if depth[stop] < g and kids:
        idx, res = node_decision(p[b, stop], q[b, stop], [tokens[b, c] for c in kids], [u_accept[b, c] for c in kids])
        assert idx is None, "the winning path stops where every candidate was rejected"
        dist = res
    return stop, dist


def sample_roots(p, q, tokens, parent, gamma, u_accept, verify_out, u_roots):
    """next_roots[b][:] = R distinct ids drawn from the stop distribution of every sequence (see above)."""
    B = p.shape[0]
    R = u_roots.shape[1]
    out = np.full((B, R), -1, dtype=np.int32)
    for b in range(B):
        _, dist = stop_distribution(p, q, tokens, parent, None if gamma is None else gamma[b], u_accept, b, verify_out)
        out[b] = sample_without_replacement(dist, u_roots[b])
    return out


# ----------------------------------------------------------------------------
# verification from next-token logits (Fig. 1 step 4; temperatures of Section 4.1)
# ----------------------------------------------------------------------------

def softmax_temperature(logits, temperature):
    """Next-token distribution exp(z_v / T) / sum_w exp(z_w / T) over the last axis, fp64, T > 0.

    Fig. 1 step 4 turns the target's next-token logits into distributions; the
    experiments sample at temperature 0.7.  The row maximum is subtracted
    before the exponential, which changes nothing mathematically.
    """
    if not temperature > 0.0:
        raise ValueError("temperature must be positive; temperature 0 is verify_tree_greedy")
    z = np.asarray(logits, dtype=np.float64) / float(temperature)
    z = z - z.max(axis=-1, keepdims=True)
    e = np.exp(z)
    return e / e.sum(axis=-1, keepdims=True)


def verify_tree_logits(target_logits, draft_logits, temperature, tokens, parent, gamma, u_accept, u_bonus, R=0,
                       trace: Optional[list] = None):
    """verify_tree on p = softmax(target_logits / T), q = softmax(draft_logits / T) (both models sample at T)."""
    p = softmax_temperature(target_logits, temperature)
    q = softmax_temperature(draft_logits, temperature)
    return verify_tree(p, q, tokens, parent, gamma, u_accept, u_bonus, R, trace)


def argmax_lowest(row):
    """Index of the largest entry; among equal largest entries the lowest id."""
    row = np.asarray(row, dtype=np.float64)
    best = 0
    for v in range(1, len(row)):
        if row[v] > row[best]:
            best = v
    return best


def verify_tree_greedy(target_logits, tokens, parent, gamma, R=0):
    """Temperature 0 (greedy sampling, Section 4.1): the target distribution is the point mass on its argmax.

    A child is accepted iff its token is the argmax of the target logits at its
    parent (min(1, p/q) is 1 there and 0 elsewhere, and the residual of a point
    mass is the same point mass); the new token at the stop node is that node's
    argmax.  No random numbers are involved.  next_roots lists the R largest
    logits of the stop node (ties: lower id first).
    """
    parent = np.asarray(parent, dtype=np.int64)
    depth, level_start = tree_levels(parent)
    n_levels = len(level_start) - 1
    N = len(parent)
    zt = np.asarray(target_logits, dtype=np.float64)
    B = zt.shape[0]
    roots = [n for n in range(N) if parent[n] < 0]
    n_roots = len(roots)
    accept_len = np.zeros(B, dtype=np.int32)
    out_tokens = np.full((B, n_levels + 1), -1, dtype=np.int32)
    out_nodes = np.full((B, n_levels), -1, dtype=np.int32)
    best_root = np.zeros(B, dtype=np.int32)
    next_roots = np.full((B, max(R, 0)), -1, dtype=np.int32)
    for b in range(B):
        g = n_levels - 1 if gamma is None else int(gamma[b])
        best = None
        for r in roots:
            u = r
            path: List[int] = []
            while depth[u] < g:
                top = argmax_lowest(zt[b, u])
                nxt = None
                for c in _children(parent, u):
                    if int(tokens[b, c]) == top:
                        nxt = c
                        break
                if nxt is None:
                    break
                path.append(nxt)
                u = nxt
            if best is None or len(path) > len(best[1]):
                best = (r, path, u)
        r, path, stop = best
        accept_len[b] = len(path)
        best_root[b] = r
        toks = ([int(tokens[b, r])] if n_roots > 1 else []) + [int(tokens[b, c]) for c in path]
        toks.append(argmax_lowest(zt[b, stop]))
        out_tokens[b, :len(toks)] = toks
        out_nodes[b, :len(path)] = path
        if R > 0:
            next_roots[b, :] = np.argsort(-zt[b, stop], kind="stable")[:R]
    return {"accept_len": accept_len, "out_tokens": out_tokens, "out_nodes": out_nodes,
            "best_root": best_root, "next_roots": next_roots}


# ----------------------------------------------------------------------------
# KV-cache update after acceptance (Fig. 1 step 6)
# ----------------------------------------------------------------------------

def commit_kv(k_cache, v_cache, k_tree, v_tree, seq_lens, accept_len, out_nodes, best_root):
    """Append the keys/values of the accepted tokens to the prefix cache (in place) and return the new lengths.

    For sequence b the committed tree tokens are the winning root (with a single root that is node 0, the last
    emitted token, whose K/V is not in the prefix yet) followed by the accepted nodes out_nodes[b][:accept_len[b]],
    written to cache rows seq_lens[b], seq_lens[b]+1, ...  Rows that would fall beyond L_max are dropped and the
    length saturates at L_max.  k_cache, v_cache: [B][H][L_max][D]; k_tree, v_tree: [B][H][N][D].
    """
    B, H, L_max, D = k_cache.shape
    new_lens = np.array(seq_lens, dtype=np.int32).copy()
    for b in range(B):
        nodes = [int(best_root[b])] + [int(n) for n in out_nodes[b][: int(accept_len[b])]]
        L = int(seq_lens[b])
        for i, n in enumerate(nodes):
            if L + i >= L_max:
                break
            k_cache[b, :, L + i, :] = k_tree[b, :, n, :]
            v_cache[b, :, L + i, :] = v_tree[b, :, n, :]
        new_lens[b] = min(L_max, L + len(nodes))
    return new_lens
