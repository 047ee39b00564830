"""Seeded synthetic inputs for tree verification in multi-candidate speculative decoding.

This module only *draws* inputs: token-tree parent arrays, query/key/value
tensors, target/draft probability rows, candidate tokens and uniforms.  It
holds none of the method's arithmetic (no mask, no attention, no accept/reject
rule), so both the CUDA library and the CPU oracle can be fed from it without
sharing any code of the method itself.

Shapes follow Llama-2-7B attention (32 heads x 128, vocabulary 32000, context
4096; Section 4.1 of the paper names the model family).  The paper's own
prompts and model weights are replaced by Gaussian tensors and Gaussian
logits: target logits ~ N(0, sigma_t^2), draft logits = target + N(0, sigma_d^2),
p and q their softmaxes, child tokens drawn i.i.d. from the draft row of the
parent (the multi-candidate sampling of Section 2.2).

All randomness comes from torch's counter-based (Philox) generators seeded as
``1000 * workload.index + 10 * layer_or_step + stream`` so any tensor can be
regenerated on its own, on either device.  Values are drawn in fp32 and rounded
once to the storage dtype; both sides then read the stored values.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, Optional, Tuple

import numpy as np
import torch

__all__ = [
    "Workload", "WORKLOADS", "workload", "parent_array", "fork_parent_array",
    "seq_lens", "gammas", "attention_inputs", "verify_inputs", "verify_logit_inputs", "UNIFORM_MARGIN",
]

# Uniforms are kept inside [UNIFORM_MARGIN, 1 - UNIFORM_MARGIN].
UNIFORM_MARGIN = 1e-4

# stream ids inside one (workload, layer/step) seed family
_S_Q, _S_KC, _S_VC, _S_KT, _S_VT = 0, 1, 2, 3, 4
_S_LOGIT_T, _S_LOGIT_D, _S_TOK, _S_UACC, _S_UBON, _S_LENS, _S_GAMMA, _S_ROOT = 0, 1, 2, 3, 4, 5, 6, 7


@dataclasses.dataclass(frozen=True)
class Workload:
    """One synthetic verification workload.

    ``n_roots`` and ``branching`` describe the token tree the way Section 4.1
    writes a k-configuration: ``n_roots`` level-0 nodes, then every node of
    level ``l`` gets ``branching[l]`` children.  ``n_roots == 1`` is the
    draft-initialised tree whose single root is the last emitted token;
    ``n_roots > 1`` is the target-initialised forest of Section 3.1.
    """
    name: str
    index: int
    dtype: str                      # "f32" or "bf16"
    B: int
    H: int
    D: int
    prefix: Tuple[int, int]         # (lo, hi) inclusive; lo == hi for a fixed prefix
    n_roots: int
    branching: Tuple[int, ...]
    gamma: Optional[Tuple[int, int]]  # per-sequence draft length range, None = full depth
    V: int
    qkv_std: float
    sigma_target: float = 3.0
    sigma_draft: float = 1.0
    n_layers: int = 1
    base_seed: Optional[int] = None
    early_stop: Optional[float] = None   # threshold beta of a synthetic early-stop process that sets gamma

    @property
    def L_max(self) -> int:
        return self.prefix[1]

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    def seed(self, layer_or_step: int, stream: int) -> int:
        base = self.base_seed if self.base_seed is not None else 1000 * self.index
        return base + 10 * layer_or_step + stream

    @property
    def n_nodes(self) -> int:
        return len(parent_array(self.n_roots, self.branching))


_INV_SQRT_128 = 1.0 / float(np.sqrt(128.0))

WORKLOADS: Dict[str, Workload] = {
    w.name: w for w in (
        Workload("tiny_fp32", 1, "f32", 1, 4, 64, (128, 128), 1, (2, 2, 2), None, 1000, 1.0, base_seed=0),
        Workload("llama7b_b1", 2, "bf16", 1, 32, 128, (512, 512), 1, (4, 2, 2, 1), None, 32000, _INV_SQRT_128),
        Workload("dynamic_slice_b8", 3, "bf16", 8, 32, 128, (2048, 2048), 1, (4, 2, 2, 1, 1, 1, 1, 1), (1, 8),
                 32000, _INV_SQRT_128),
        Workload("long_context_b16", 4, "bf16", 16, 32, 128, (4096, 4096), 1, (4, 2, 2, 1), None, 32000,
                 _INV_SQRT_128, n_layers=32),
        Workload("target_init_b32", 5, "bf16", 32, 32, 128, (256, 4096), 8, (1, 2, 2, 1, 1, 1), (1, 6), 32000,
                 _INV_SQRT_128, sigma_draft=1.5),
        # the paper's own tree shapes (Section 4.1): the static target-initialised configuration (2; 4,3,1,1) and
        # the fork of width 16 and depth 5 hanging off the last emitted token, cut by an early stop (beta = 0.4)
        Workload("paper_static_2_4_3_1_1", 6, "bf16", 16, 32, 128, (512, 2048), 2, (4, 3, 1, 1), None, 32000,
                 _INV_SQRT_128),
        Workload("paper_fork_w16_d5", 7, "bf16", 16, 32, 128, (512, 2048), 1, (16, 1, 1, 1, 1), (1, 5), 32000,
                 _INV_SQRT_128, early_stop=0.4),
    )
}


def workload(name_or_index) -> Workload:
    if isinstance(name_or_index, int):
        for w in WORKLOADS.values():
            if w.index == name_or_index:
                return w
        raise KeyError(name_or_index)
    return WORKLOADS[name_or_index]


def parent_array(n_roots: int, branching) -> np.ndarray:
    """Parent index of every node of a k-configuration tree, nodes in level (BFS) order.

    Roots carry -1 (their parent is the end of the prefix).  Children of one
    node are contiguous and follow the order of their parents.
    """
    if n_roots < 1:
        raise ValueError("n_roots must be >= 1")
    parent = [-1] * n_roots
    level = list(range(n_roots))
    for k in branching:
        if k < 1:
            raise ValueError("branching factors must be >= 1")
        nxt = []
        for u in level:
            for _ in range(k):
                nxt.append(len(parent))
                parent.append(u)
        level = nxt
    return np.asarray(parent, dtype=np.int32)


def fork_parent_array(width: int, depth: int) -> np.ndarray:
    """Fork-shaped tree of Section 3.2: ``width`` chains that never re-branch, ``depth`` nodes each."""
    return parent_array(width, (1,) * (depth - 1))


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def seq_lens(w: Workload, step: int = 0) -> np.ndarray:
    """Prefix length of every sequence (int32[B])."""
    lo, hi = w.prefix
    if lo == hi:
        return np.full(w.B, lo, dtype=np.int32)
    g = _gen("cpu", w.seed(step, _S_LENS))
    return torch.randint(lo, hi + 1, (w.B,), generator=g).numpy().astype(np.int32)


def gammas(w: Workload, step: int = 0) -> np.ndarray:
    """Draft length gamma kept for every sequence at this step (int32[B]); full depth if the workload is static."""
    full = len(w.branching)
    if w.gamma is None:
        return np.full(w.B, full, dtype=np.int32)
    lo, hi = w.gamma
    g = _gen("cpu", w.seed(step, _S_GAMMA))
    if w.early_stop is not None:
        return _early_stop_gammas(w, g, lo, hi)
    return torch.randint(lo, hi + 1, (w.B,), generator=g).numpy().astype(np.int32)


def _early_stop_gammas(w: Workload, g: torch.Generator, lo: int, hi: int) -> np.ndarray:
    """Stand-in for the decision model of Section 3.3, which is not part of the verification path.

    Every draft turn gives each of the W candidate sequences a score in (0, 1) (here uniform); a sequence's
    predicted chance of being accepted so far is the product of its scores; drafting stops after the first turn
    at which every sequence is below the threshold, else at the maximum depth.  gamma = turns drafted.
    """
    W = w.n_roots if w.n_roots > 1 else w.branching[0]
    score = torch.rand((w.B, hi, W), generator=g, dtype=torch.float64).cumprod(dim=1)
    alive = (score.max(dim=2).values >= w.early_stop).numpy()          # [B][turn]
    out = np.full(w.B, hi, dtype=np.int32)
    for b in range(w.B):
        for t in range(hi):
            if not alive[b, t]:
                out[b] = t + 1
                break
    return np.clip(out, lo, hi).astype(np.int32)


def attention_inputs(w: Workload, layer: int = 0, device="cpu", std: Optional[float] = None):
    """q, k_cache, v_cache, k_tree, v_tree for one layer.

    Layouts: q, k_tree, v_tree ``[B][H][N][D]``; k_cache, v_cache ``[B][H][L_max][D]``.
    ``std`` overrides the workload's value scale (used for sharp-softmax cases).
    """
    s = w.qkv_std if std is None else std
    N = w.n_nodes
    dt = w.torch_dtype

    def draw(shape, stream):
        g = _gen(device, w.seed(layer, stream))
        x = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
        return (x * s).to(dt)

    return {
        "q": draw((w.B, w.H, N, w.D), _S_Q),
        "k_cache": draw((w.B, w.H, w.L_max, w.D), _S_KC),
        "v_cache": draw((w.B, w.H, w.L_max, w.D), _S_VC),
        "k_tree": draw((w.B, w.H, N, w.D), _S_KT),
        "v_tree": draw((w.B, w.H, N, w.D), _S_VT),
    }


def verify_inputs(w: Workload, step: int = 0, device="cpu", parent: Optional[np.ndarray] = None,
                  B: Optional[int] = None, V: Optional[int] = None):
    """p, q ``[B][N][V]`` fp32 probabilities, tokens ``[B][N]`` int32, u_accept, u_bonus ``[B][N]`` fp32.

    Row n of p (q) is the target (draft) next-token distribution after node n.
    A non-root node's token is an independent draw from its parent's q row.
    With one root the root token is an arbitrary id (the last emitted token);
    with several roots they are the ``n_roots`` most probable ids of one more
    target row (Section 3.1: the target proposes the first level itself).
    """
    if parent is None:
        parent = parent_array(w.n_roots, w.branching)
    B = w.B if B is None else B
    V = w.V if V is None else V
    N = len(parent)
    n_roots = int((parent < 0).sum())

    gt = _gen(device, w.seed(step, _S_LOGIT_T))
    gd = _gen(device, w.seed(step, _S_LOGIT_D))
    logit_t = torch.randn((B, N, V), generator=gt, device=device, dtype=torch.float32) * w.sigma_target
    logit_d = logit_t + torch.randn((B, N, V), generator=gd, device=device, dtype=torch.float32) * w.sigma_draft
    p = torch.softmax(logit_t, dim=-1)
    del logit_t
    q = torch.softmax(logit_d, dim=-1)
    del logit_d

    gk = _gen(device, w.seed(step, _S_TOK))
    tokens = torch.zeros((B, N), dtype=torch.int64, device=device)
    if n_roots == 1:
        tokens[:, 0] = torch.randint(0, V, (B,), generator=gk, device=device)
    else:
        gr = _gen(device, w.seed(step, _S_ROOT))
        root_row = torch.softmax(torch.randn((B, V), generator=gr, device=device) * w.sigma_target, dim=-1)
        tokens[:, :n_roots] = torch.topk(root_row, n_roots, dim=-1).indices
    # children of node u are the contiguous run of nodes whose parent is u
    u = 0
    c = n_roots
    while c < N:
        u = int(parent[c])
        e = c
        while e < N and parent[e] == u:
            e += 1
        tokens[:, c:e] = torch.multinomial(q[:, u, :], e - c, replacement=True, generator=gk)
        c = e

    ga = _gen(device, w.seed(step, _S_UACC))
    gb = _gen(device, w.seed(step, _S_UBON))
    lo, hi = UNIFORM_MARGIN, 1.0 - UNIFORM_MARGIN
    u_accept = torch.rand((B, N), generator=ga, device=device, dtype=torch.float32).clamp_(lo, hi)
    u_bonus = torch.rand((B, N), generator=gb, device=device, dtype=torch.float32).clamp_(lo, hi)
    return {"p": p, "q": q, "tokens": tokens.to(torch.int32), "u_accept": u_accept, "u_bonus": u_bonus}


def verify_logit_inputs(w: Workload, temperature: float, dtype=torch.float32, step: int = 0, device="cpu",
                        parent: Optional[np.ndarray] = None, B: Optional[int] = None, V: Optional[int] = None):
    """target_logits, draft_logits ``[B][N][V]`` in `dtype`, tokens ``[B][N]`` int32, u_accept, u_bonus ``[B][N]`` fp32.

    The logits are those behind ``verify_inputs`` (draft = target + noise), rounded to `dtype`.  What the draft
    proposes depends on how it samples: at temperature > 0 a node's children are independent draws from
    softmax(draft logits of the parent / temperature); at temperature 0 they are the parent's largest draft
    logits, one per child.  Roots are as in ``verify_inputs``.
    """
    if parent is None:
        parent = parent_array(w.n_roots, w.branching)
    B = w.B if B is None else B
    V = w.V if V is None else V
    N = len(parent)
    n_roots = int((parent < 0).sum())

    gt = _gen(device, w.seed(step, _S_LOGIT_T))
    gd = _gen(device, w.seed(step, _S_LOGIT_D))
    logit_t = torch.randn((B, N, V), generator=gt, device=device, dtype=torch.float32) * w.sigma_target
    logit_d = logit_t + torch.randn((B, N, V), generator=gd, device=device, dtype=torch.float32) * w.sigma_draft
    logit_t = logit_t.to(dtype)
    logit_d = logit_d.to(dtype)

    gk = _gen(device, w.seed(step, _S_TOK))
    tokens = torch.zeros((B, N), dtype=torch.int64, device=device)
    if n_roots == 1:
        tokens[:, 0] = torch.randint(0, V, (B,), generator=gk, device=device)
    else:
        gr = _gen(device, w.seed(step, _S_ROOT))
        root_row = torch.randn((B, V), generator=gr, device=device) * w.sigma_target
        tokens[:, :n_roots] = torch.topk(root_row, n_roots, dim=-1).indices
    c = n_roots
    while c < N:
        u = int(parent[c])
        e = c
        while e < N and parent[e] == u:
            e += 1
        row = logit_d[:, u, :].float()
        if temperature > 0:
            tokens[:, c:e] = torch.multinomial(torch.softmax(row / temperature, dim=-1), e - c, replacement=True,
                                               generator=gk)
        else:
            tokens[:, c:e] = torch.topk(row, e - c, dim=-1).indices
        c = e

    ga = _gen(device, w.seed(step, _S_UACC))
    gb = _gen(device, w.seed(step, _S_UBON))
    lo, hi = UNIFORM_MARGIN, 1.0 - UNIFORM_MARGIN
    u_accept = torch.rand((B, N), generator=ga, device=device, dtype=torch.float32).clamp_(lo, hi)
    u_bonus = torch.rand((B, N), generator=gb, device=device, dtype=torch.float32).clamp_(lo, hi)
    return {"target_logits": logit_t, "draft_logits": logit_d, "tokens": tokens.to(torch.int32),
            "u_accept": u_accept, "u_bonus": u_bonus}
