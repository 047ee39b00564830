"""ctypes binding of libmcsd.so: argument marshalling only.

Tensors are torch tensors on a CUDA device (torch supplies memory and streams); every function
passes raw pointers and sizes to the C entry point of the same name (include/mcsd.h) on torch's
current stream and raises McsdError on a non-zero status.
"""
from __future__ import annotations

import ctypes
import os
from typing import NamedTuple, Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# MCSD_LIB selects another build of the same library (A/B timing of kernel variants)
_LIB_PATH = os.environ.get("MCSD_LIB") or os.path.join(_HERE, "libmcsd.so")

MCSD_BF16 = 0
MCSD_F32 = 1
MCSD_MAX_NODES = 192
MCSD_MAX_WORDS = 3

_EXPORTS = (
    "mcsd_status_string", "mcsd_last_cuda_error", "mcsd_launch_count", "mcsd_build_mask", "mcsd_tree_attention_workspace_bytes",
    "mcsd_tree_attention", "mcsd_tree_attention_gqa", "mcsd_workspace_status", "verify_node_states", "mcsd_tree_attention_path", "mcsd_tree_attention_plan", "mcsd_selftest_bounded_wait", "mcsd_verify_tree_workspace_bytes", "mcsd_verify_tree", "mcsd_verify_tree_logits", "mcsd_verify_tree_static", "mcsd_commit_kv", "mcsd_sample_roots",
    "mcsd_sample_roots_logits", "mcsd_verify_shard_workspace_bytes", "mcsd_verify_shard_gather", "mcsd_verify_shard_round",
    "mcsd_verify_shard_select", "mcsd_verify_shard_pick",
)


def _load() -> ctypes.CDLL:
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(
            "libmcsd.so is not built (%s missing). Build it with `python -m paper_2409_10644_b200.build`; "
            "there is no fallback path." % _LIB_PATH)
    lib = ctypes.CDLL(_LIB_PATH)
    c_int, c_void_p, c_size_t, c_float = ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_float
    lib.mcsd_status_string.restype = ctypes.c_char_p
    lib.mcsd_status_string.argtypes = [c_int]
    lib.mcsd_last_cuda_error.restype = c_int
    lib.mcsd_last_cuda_error.argtypes = []
    lib.mcsd_launch_count.restype = ctypes.c_longlong
    lib.mcsd_launch_count.argtypes = []
    lib.mcsd_build_mask.restype = c_int
    lib.mcsd_build_mask.argtypes = [c_void_p, c_int, c_void_p, c_int, c_void_p, c_void_p, c_void_p,
                                    ctypes.POINTER(c_int), c_void_p]
    lib.mcsd_tree_attention_workspace_bytes.restype = c_size_t
    lib.mcsd_tree_attention_workspace_bytes.argtypes = [c_int] * 6
    lib.mcsd_selftest_bounded_wait.restype = c_int
    lib.mcsd_selftest_bounded_wait.argtypes = [c_void_p, c_size_t, c_int, c_void_p]
    lib.mcsd_tree_attention_path.restype = c_int
    lib.mcsd_tree_attention_path.argtypes = [c_int] * 7
    lib.mcsd_tree_attention_plan.restype = c_int
    lib.mcsd_tree_attention_plan.argtypes = [c_int] * 7 + [c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_int, c_void_p, c_void_p]
    lib.mcsd_tree_attention.restype = c_int
    lib.mcsd_tree_attention.argtypes = [c_void_p] * 9 + [c_int] * 6 + [c_float, c_int, c_void_p, c_size_t, c_void_p]
    lib.mcsd_tree_attention_gqa.restype = c_int
    lib.mcsd_tree_attention_gqa.argtypes = [c_void_p] * 9 + [c_int] * 7 + [c_float, c_int, c_void_p, c_size_t, c_void_p]
    lib.mcsd_workspace_status.restype = c_int
    lib.mcsd_workspace_status.argtypes = [c_void_p, c_void_p]
    lib.mcsd_verify_tree_workspace_bytes.restype = c_size_t
    lib.mcsd_verify_tree_workspace_bytes.argtypes = [c_int] * 3
    lib.mcsd_verify_tree.restype = c_int
    lib.mcsd_verify_tree.argtypes = ([c_void_p] * 5 + [c_int, c_int] + [c_void_p] * 3 + [c_int] * 3 +
                                     [c_void_p] * 5 + [c_int, c_void_p, c_size_t, c_void_p])
    lib.mcsd_verify_tree_logits.restype = c_int
    lib.mcsd_verify_tree_logits.argtypes = ([c_void_p, c_void_p, c_int, c_float] + [c_void_p] * 3 + [c_int, c_int] +
                                            [c_void_p] * 3 + [c_int] * 3 + [c_void_p] * 5 +
                                            [c_int, c_void_p, c_size_t, c_void_p])
    lib.mcsd_sample_roots.restype = c_int
    lib.mcsd_sample_roots.argtypes = [c_void_p] * 5 + [c_int, c_void_p] + [c_int] * 4 + [c_void_p, c_void_p, c_size_t, c_void_p]
    lib.mcsd_sample_roots_logits.restype = c_int
    lib.mcsd_sample_roots_logits.argtypes = ([c_void_p, c_void_p, c_int, c_float] + [c_void_p] * 3 + [c_int, c_void_p] +
                                             [c_int] * 4 + [c_void_p, c_void_p, c_size_t, c_void_p])
    lib.mcsd_verify_tree_static.restype = c_int
    lib.mcsd_verify_tree_static.argtypes = ([c_void_p] * 5 + [c_int, c_int] + [c_void_p] * 3 + [c_int] * 3 +
                                            [c_void_p] * 5 + [c_int, c_void_p])
    lib.mcsd_commit_kv.restype = c_int
    lib.mcsd_commit_kv.argtypes = [c_void_p] * 4 + [c_int] + [c_void_p] * 4 + [c_int] * 7 + [c_void_p]
    lib.mcsd_verify_shard_workspace_bytes.restype = c_size_t
    lib.mcsd_verify_shard_workspace_bytes.argtypes = [c_int] * 2
    lib.mcsd_verify_shard_gather.restype = c_int
    lib.mcsd_verify_shard_gather.argtypes = [c_void_p] * 5 + [c_int, c_void_p] + [c_int] * 5 + [c_void_p, c_void_p]
    lib.mcsd_verify_shard_round.restype = c_int
    lib.mcsd_verify_shard_round.argtypes = ([c_void_p] * 4 + [c_int] + [c_void_p] * 4 + [c_int] * 4 +
                                            [c_void_p, c_size_t, c_void_p])
    lib.mcsd_verify_shard_select.restype = c_int
    lib.mcsd_verify_shard_select.argtypes = ([c_void_p] * 3 + [c_int] * 9 + [c_void_p] * 5 +
                                             [c_void_p, c_size_t, c_void_p])
    lib.mcsd_verify_shard_pick.restype = c_int
    lib.mcsd_verify_shard_pick.argtypes = ([c_void_p] * 3 + [c_int] * 8 + [c_void_p] * 2 +
                                           [c_void_p, c_size_t, c_void_p])
    return lib


lib = _load()


class McsdError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib.mcsd_status_string(status).decode()
        if status == -6:
            msg += " (cudaError %d)" % lib.mcsd_last_cuda_error()
        super().__init__("%s: %s [%d]" % (where, msg, status))


def mcsd_status_string(status: int) -> str:
    return lib.mcsd_status_string(int(status)).decode()


def mcsd_launch_count() -> int:
    return int(lib.mcsd_launch_count())


def _check(status: int, where: str):
    if status != 0:
        raise McsdError(status, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dev_tensor(t: torch.Tensor, dtype, name: str) -> torch.Tensor:
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise ValueError("%s must be a contiguous CUDA tensor of dtype %s" % (name, dtype))
    return t


class TreeMask(NamedTuple):
    """Outputs of mcsd_build_mask plus the device copy of the parent array the verify step needs."""
    anc: torch.Tensor            # uint64 bit patterns stored as int64 [N][words]
    depth: torch.Tensor          # int32 [N]
    level_start: torch.Tensor    # int32 [N + 1] (first n_levels + 1 entries valid)
    level_start_host: np.ndarray  # int32 [n_levels + 1]
    parent: torch.Tensor         # int32 [N]
    n_nodes: int
    n_levels: int
    n_roots: int
    words: int


def mcsd_build_mask(parent, device="cuda", words: Optional[int] = None) -> TreeMask:
    """Ancestor bitsets, depths and level starts of a level-ordered token tree (built once per tree shape)."""
    parent = np.ascontiguousarray(np.asarray(parent, dtype=np.int32))
    n = int(parent.shape[0])
    if words is None:
        words = max(1, (n + 63) // 64)
    dev = torch.device(device)
    anc = torch.zeros((max(n, 1), words), dtype=torch.int64, device=dev)
    depth = torch.zeros(max(n, 1), dtype=torch.int32, device=dev)
    level_start = torch.zeros(max(n, 1) + 1, dtype=torch.int32, device=dev)
    ls_host = np.zeros(max(n, 1) + 1, dtype=np.int32)
    n_levels = ctypes.c_int(0)
    with torch.cuda.device(dev):
        st = lib.mcsd_build_mask(parent.ctypes.data_as(ctypes.c_void_p), n, _ptr(anc), words, _ptr(depth),
                                 _ptr(level_start), ls_host.ctypes.data_as(ctypes.c_void_p),
                                 ctypes.byref(n_levels), _stream())
    _check(st, "mcsd_build_mask")
    parent_dev = torch.from_numpy(parent).to(dev)
    return TreeMask(anc, depth, level_start, ls_host[: n_levels.value + 1].copy(), parent_dev, n, n_levels.value,
                    int((parent < 0).sum()), words)


def n_active_from_gamma(level_start_host, gamma) -> np.ndarray:
    """Dynamic sliced mask as a row count: keeping gamma draft levels keeps level_start[gamma + 1] nodes."""
    ls = np.asarray(level_start_host)
    g = np.clip(np.asarray(gamma, dtype=np.int64), 0, len(ls) - 2)
    return ls[g + 1].astype(np.int32)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return MCSD_BF16
    if t.dtype == torch.float32:
        return MCSD_F32
    raise ValueError("tree attention takes bf16 or fp32 tensors")


def mcsd_tree_attention_workspace_bytes(B, H, N, D, L_max, dtype) -> int:
    return int(lib.mcsd_tree_attention_workspace_bytes(B, H, N, D, L_max, dtype))


def verify_node_states(workspace: torch.Tensor, B: int, N: int):
    """Views of what the verify call left per (sequence, node) in its workspace: `next_child` int32[B][N] (accepted
    child or -1) and `c` float64[B][N] (the stop distribution at that node is max(p - c q, 0))."""
    raw = workspace[256:256 + 16 * B * N]
    return {"next_child": raw.view(torch.int32).view(B, N, 4)[..., 0], "c": raw.view(torch.float64).view(B, N, 2)[..., 1]}


def mcsd_selftest_bounded_wait(workspace: torch.Tensor, microseconds: int = 1000) -> None:
    """Launches the bounded-wait self-test on `workspace` (see mcsd.h); mcsd_workspace_status(workspace) then reads
    MCSD_ERR_TIMEOUT and the workspace has to be zero-filled again."""
    _dev_tensor(workspace, torch.uint8, "workspace")
    with torch.cuda.device(workspace.device):
        st = lib.mcsd_selftest_bounded_wait(_ptr(workspace), workspace.numel(), int(microseconds), _stream())
    _check(st, "mcsd_selftest_bounded_wait")


def mcsd_tree_attention_path(B, H_q, H_kv, N, D, L_max, dtype_code) -> int:
    """1 if the tensor-core kernel takes this shape, 0 if the CUDA-core kernel does (see mcsd.h); raises on bad shapes."""
    st = int(lib.mcsd_tree_attention_path(B, H_q, H_kv, N, D, L_max, dtype_code))
    if st < 0:
        _check(st, "mcsd_tree_attention_path")
    return st


def mcsd_tree_attention_plan(B, H_q, H_kv, N, D, L_max, dtype_code, seq_lens, n_active=None, n_blocks=148, probe_tiles=()):
    """How the tensor-core kernel cuts a launch among ``n_blocks`` thread blocks (host only, see mcsd.h).

    ``seq_lens`` / ``n_active``: host int32 arrays.  Returns ``(blocks_used, first_tile[n_blocks + 1], info[4],
    probe_out[len(probe_tiles)][8])`` as numpy arrays.
    """
    import numpy as np
    lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    if lens.shape != (B,):
        raise ValueError("seq_lens must have B entries")
    nact = None if n_active is None else np.ascontiguousarray(n_active, dtype=np.int32)
    if nact is not None and nact.shape != (B,):
        raise ValueError("n_active must have B entries")
    if not 1 <= int(n_blocks) <= 160:
        raise ValueError("n_blocks must be 1..160")
    probes = np.ascontiguousarray(probe_tiles, dtype=np.int64).reshape(-1)
    first = np.zeros(int(n_blocks) + 1, dtype=np.int64)
    info = np.zeros(4, dtype=np.int64)
    out = np.zeros((len(probes), 8), dtype=np.int64)
    st = int(lib.mcsd_tree_attention_plan(B, H_q, H_kv, N, D, L_max, dtype_code, lens.ctypes.data,
                                          None if nact is None else nact.ctypes.data, int(n_blocks), first.ctypes.data,
                                          info.ctypes.data, len(probes), probes.ctypes.data if len(probes) else None,
                                          out.ctypes.data if len(probes) else None))
    if st < 0:
        _check(st, "mcsd_tree_attention_plan")
    return st, first, info, out


def new_workspace(nbytes: int, device) -> torch.Tensor:
    """Zero-filled, 256-byte aligned scratch buffer (torch's allocator aligns to 512 bytes)."""
    return torch.zeros(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def mcsd_tree_attention(q, k_cache, v_cache, k_tree, v_tree, seq_lens, n_active, mask: TreeMask,
                        out: Optional[torch.Tensor] = None, softmax_scale: Optional[float] = None,
                        workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """out[b][h][n] = attention of tree token n over the prefix cache and its root path (see mcsd.h).

    Key/value tensors with fewer heads than q select grouped-query attention (query head h reads head h // G)."""
    dt = q.dtype
    B, H, N, D = q.shape
    L_max = k_cache.shape[2]
    H_kv = k_tree.shape[1]
    if H_kv < 1 or H % H_kv:
        raise ValueError("q has %d heads, the key/value tensors %d" % (H, H_kv))
    for name, t, shape in (("q", q, (B, H, N, D)), ("k_cache", k_cache, (B, H_kv, L_max, D)),
                           ("v_cache", v_cache, (B, H_kv, L_max, D)), ("k_tree", k_tree, (B, H_kv, N, D)),
                           ("v_tree", v_tree, (B, H_kv, N, D))):
        _dev_tensor(t, dt, name)
        if tuple(t.shape) != shape:
            raise ValueError("%s has shape %s, expected %s" % (name, tuple(t.shape), shape))
    _dev_tensor(seq_lens, torch.int32, "seq_lens")
    if n_active is not None:
        _dev_tensor(n_active, torch.int32, "n_active")
    if mask.n_nodes != N:
        raise ValueError("mask was built for %d nodes, q has %d" % (mask.n_nodes, N))
    if out is None:
        out = torch.empty_like(q)
    code = _dtype_code(q)
    if softmax_scale is None:
        softmax_scale = 1.0 / float(np.sqrt(D))
    need = mcsd_tree_attention_workspace_bytes(B, H, N, D, L_max, code)
    if workspace is None:
        workspace = new_workspace(need, q.device)
    with torch.cuda.device(q.device):
        if H_kv == H:
            st = lib.mcsd_tree_attention(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(k_tree), _ptr(v_tree), _ptr(out),
                                         _ptr(seq_lens), _ptr(n_active), _ptr(mask.anc), mask.words, B, H, N, D, L_max,
                                         ctypes.c_float(softmax_scale), code, _ptr(workspace), workspace.numel(),
                                         _stream())
        else:
            st = lib.mcsd_tree_attention_gqa(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(k_tree), _ptr(v_tree), _ptr(out),
                                             _ptr(seq_lens), _ptr(n_active), _ptr(mask.anc), mask.words, B, H, H_kv, N, D,
                                             L_max, ctypes.c_float(softmax_scale), code, _ptr(workspace),
                                             workspace.numel(), _stream())
    _check(st, "mcsd_tree_attention")
    return out


def mcsd_workspace_status(workspace: torch.Tensor) -> int:
    with torch.cuda.device(workspace.device):
        return int(lib.mcsd_workspace_status(_ptr(workspace), _stream()))


def mcsd_verify_tree_workspace_bytes(B, N, V) -> int:
    return int(lib.mcsd_verify_tree_workspace_bytes(B, N, V))


def mcsd_verify_tree(p, q, tokens, mask: TreeMask, gamma, u_accept, u_bonus, R: int = 0,
                     workspace: Optional[torch.Tensor] = None, out: Optional[dict] = None) -> dict:
    """Accept/reject walk, longest-path selection and new-token sampling (see mcsd.h). Returns device tensors."""
    B, N, V = p.shape
    _dev_tensor(p, torch.float32, "p")
    _dev_tensor(q, torch.float32, "q")
    _dev_tensor(tokens, torch.int32, "tokens")
    _dev_tensor(u_accept, torch.float32, "u_accept")
    _dev_tensor(u_bonus, torch.float32, "u_bonus")
    if gamma is not None:
        _dev_tensor(gamma, torch.int32, "gamma")
    if mask.n_nodes != N or tuple(q.shape) != (B, N, V) or tuple(tokens.shape) != (B, N):
        raise ValueError("shape mismatch between p, q, tokens and the tree")
    dev = p.device
    nl = mask.n_levels
    if out is None:
        out = {
            "accept_len": torch.empty(B, dtype=torch.int32, device=dev),
            "out_tokens": torch.empty((B, nl + 1), dtype=torch.int32, device=dev),
            "out_nodes": torch.empty((B, nl), dtype=torch.int32, device=dev),
            "best_root": torch.empty(B, dtype=torch.int32, device=dev),
            "next_roots": torch.empty((B, R), dtype=torch.int32, device=dev) if R > 0 else None,
        }
    if workspace is None:
        workspace = new_workspace(mcsd_verify_tree_workspace_bytes(B, N, V), dev)
    with torch.cuda.device(dev):
        st = lib.mcsd_verify_tree(_ptr(p), _ptr(q), _ptr(tokens), _ptr(mask.parent), _ptr(mask.level_start), nl,
                                  mask.n_roots, _ptr(gamma), _ptr(u_accept), _ptr(u_bonus), B, N, V,
                                  _ptr(out["accept_len"]), _ptr(out["out_tokens"]), _ptr(out["out_nodes"]),
                                  _ptr(out["best_root"]), _ptr(out.get("next_roots")), R, _ptr(workspace),
                                  workspace.numel(), _stream())
    _check(st, "mcsd_verify_tree")
    return out


def mcsd_verify_tree_logits(target_logits, draft_logits, temperature: float, tokens, mask: TreeMask, gamma,
                            u_accept, u_bonus, R: int = 0, workspace: Optional[torch.Tensor] = None,
                            out: Optional[dict] = None) -> dict:
    """mcsd_verify_tree on softmax(logits / temperature), formed inside the kernels; temperature 0 is greedy
    verification, for which draft_logits, u_accept and u_bonus may be None (see mcsd.h)."""
    B, N, V = target_logits.shape
    dt = target_logits.dtype
    if dt not in (torch.float32, torch.bfloat16):
        raise ValueError("logits must be float32 or bfloat16")
    _dev_tensor(target_logits, dt, "target_logits")
    _dev_tensor(tokens, torch.int32, "tokens")
    if draft_logits is not None:
        _dev_tensor(draft_logits, dt, "draft_logits")
        if tuple(draft_logits.shape) != (B, N, V):
            raise ValueError("shape mismatch between target and draft logits")
    if u_accept is not None:
        _dev_tensor(u_accept, torch.float32, "u_accept")
    if u_bonus is not None:
        _dev_tensor(u_bonus, torch.float32, "u_bonus")
    if gamma is not None:
        _dev_tensor(gamma, torch.int32, "gamma")
    if mask.n_nodes != N or tuple(tokens.shape) != (B, N):
        raise ValueError("shape mismatch between logits, tokens and the tree")
    dev = target_logits.device
    nl = mask.n_levels
    if out is None:
        out = {
            "accept_len": torch.empty(B, dtype=torch.int32, device=dev),
            "out_tokens": torch.empty((B, nl + 1), dtype=torch.int32, device=dev),
            "out_nodes": torch.empty((B, nl), dtype=torch.int32, device=dev),
            "best_root": torch.empty(B, dtype=torch.int32, device=dev),
            "next_roots": torch.empty((B, R), dtype=torch.int32, device=dev) if R > 0 else None,
        }
    if workspace is None:
        workspace = new_workspace(mcsd_verify_tree_workspace_bytes(B, N, V), dev)
    code = MCSD_BF16 if dt == torch.bfloat16 else MCSD_F32
    with torch.cuda.device(dev):
        st = lib.mcsd_verify_tree_logits(_ptr(target_logits), _ptr(draft_logits), code, float(temperature), _ptr(tokens),
                                         _ptr(mask.parent), _ptr(mask.level_start), nl, mask.n_roots, _ptr(gamma),
                                         _ptr(u_accept), _ptr(u_bonus), B, N, V, _ptr(out["accept_len"]),
                                         _ptr(out["out_tokens"]), _ptr(out["out_nodes"]), _ptr(out["best_root"]),
                                         _ptr(out.get("next_roots")), R, _ptr(workspace), workspace.numel(), _stream())
    _check(st, "mcsd_verify_tree_logits")
    return out


def mcsd_sample_roots(p, q, verify_out: dict, mask: TreeMask, u_roots, workspace: torch.Tensor,
                      temperature: Optional[float] = None, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """R distinct new tokens per sequence from the distribution the winning path stopped with (see mcsd.h).

    `p`, `q` are the probability rows given to mcsd_verify_tree, or -- with `temperature` -- the target and draft
    logits given to mcsd_verify_tree_logits; `verify_out` and `workspace` are that call's results and workspace."""
    B, N, V = p.shape
    _dev_tensor(u_roots, torch.float32, "u_roots")
    R = int(u_roots.shape[1])
    if out is None:
        out = torch.empty((B, R), dtype=torch.int32, device=p.device)
    args = (_ptr(verify_out["accept_len"]), _ptr(verify_out["out_nodes"]), _ptr(verify_out["best_root"]), mask.n_levels,
            _ptr(u_roots), B, N, V, R, _ptr(out), _ptr(workspace), workspace.numel(), _stream())
    with torch.cuda.device(p.device):
        if temperature is None:
            _dev_tensor(p, torch.float32, "p")
            _dev_tensor(q, torch.float32, "q")
            st = lib.mcsd_sample_roots(_ptr(p), _ptr(q), *args)
        else:
            code = MCSD_BF16 if p.dtype == torch.bfloat16 else MCSD_F32
            _dev_tensor(p, p.dtype, "target_logits")
            _dev_tensor(q, p.dtype, "draft_logits")
            st = lib.mcsd_sample_roots_logits(_ptr(p), _ptr(q), code, float(temperature), *args)
    _check(st, "mcsd_sample_roots")
    return out


def mcsd_verify_tree_static(p, q, tokens, mask: TreeMask, gamma, u_accept, u_bonus, out: dict, R: int = 0) -> dict:
    """mcsd_verify_tree without a workspace, for callers that cannot allocate device memory at call time.

    The scratch is a fixed array inside the library (B * N <= 16384 node states); `out` must hold the
    preallocated result tensors (accept_len, out_tokens, out_nodes, best_root, next_roots), so this wrapper
    allocates nothing either.  Calls share the array: do not let two of them overlap on the GPU."""
    B, N, V = p.shape
    # the same argument checks as mcsd_verify_tree (none of them allocates), plus the caller's result tensors
    _dev_tensor(p, torch.float32, "p")
    _dev_tensor(q, torch.float32, "q")
    _dev_tensor(tokens, torch.int32, "tokens")
    _dev_tensor(u_accept, torch.float32, "u_accept")
    _dev_tensor(u_bonus, torch.float32, "u_bonus")
    if gamma is not None:
        _dev_tensor(gamma, torch.int32, "gamma")
        if tuple(gamma.shape) != (B,):
            raise ValueError("gamma must have one entry per sequence")
    if (mask.n_nodes != N or tuple(q.shape) != (B, N, V) or tuple(tokens.shape) != (B, N) or
            tuple(u_accept.shape) != (B, N) or tuple(u_bonus.shape) != (B, N)):
        raise ValueError("shape mismatch between p, q, tokens, the uniforms and the tree")
    nl = mask.n_levels
    want = {"accept_len": (B,), "out_tokens": (B, nl + 1), "out_nodes": (B, nl), "best_root": (B,)}
    if R > 0:
        want["next_roots"] = (B, R)
    for name, shape in want.items():
        t = out.get(name)
        if t is None:
            raise ValueError("out[%r] is missing" % name)
        _dev_tensor(t, torch.int32, "out[%r]" % name)
        if tuple(t.shape) != shape:
            raise ValueError("out[%r] must have shape %r" % (name, shape))
    with torch.cuda.device(p.device):
        st = lib.mcsd_verify_tree_static(_ptr(p), _ptr(q), _ptr(tokens), _ptr(mask.parent), _ptr(mask.level_start),
                                         mask.n_levels, mask.n_roots, _ptr(gamma), _ptr(u_accept), _ptr(u_bonus),
                                         B, N, V, _ptr(out["accept_len"]), _ptr(out["out_tokens"]),
                                         _ptr(out["out_nodes"]), _ptr(out["best_root"]), _ptr(out.get("next_roots")),
                                         R, _stream())
    _check(st, "mcsd_verify_tree_static")
    return out


def layer_pointer_table(tensors) -> torch.Tensor:
    """Device array of the data pointers of per-layer tensors (int64), as mcsd_commit_kv takes them."""
    dev = tensors[0].device
    return torch.tensor([t.data_ptr() for t in tensors], dtype=torch.int64, device=dev)


def mcsd_commit_kv(k_cache_ptrs, v_cache_ptrs, k_tree_ptrs, v_tree_ptrs, seq_lens, verify_out, mask: TreeMask,
                   B: int, H: int, D: int, L_max: int, dtype: torch.dtype) -> None:
    """Append the accepted tokens' K/V to every layer's prefix cache and grow seq_lens (see mcsd.h).

    The four `*_ptrs` arguments are device int64 tensors from layer_pointer_table(); `verify_out` is the dict
    returned by mcsd_verify_tree."""
    n_layers = int(k_cache_ptrs.numel())
    code = MCSD_BF16 if dtype == torch.bfloat16 else MCSD_F32
    _dev_tensor(seq_lens, torch.int32, "seq_lens")
    with torch.cuda.device(seq_lens.device):
        st = lib.mcsd_commit_kv(_ptr(k_cache_ptrs), _ptr(v_cache_ptrs), _ptr(k_tree_ptrs), _ptr(v_tree_ptrs), n_layers,
                                _ptr(seq_lens), _ptr(verify_out["accept_len"]), _ptr(verify_out["out_nodes"]),
                                _ptr(verify_out["best_root"]), mask.n_levels, B, H, mask.n_nodes, D, L_max, code,
                                _stream())
    _check(st, "mcsd_commit_kv")


def mcsd_verify_shard_workspace_bytes(B, N) -> int:
    return int(lib.mcsd_verify_shard_workspace_bytes(B, N))


class VocabShard:
    """One rank's tensors and calls of the vocabulary-sharded verify step (see mcsd.h): p_shard / q_shard hold
    columns [v0, v0 + Vs) of the two probability tensors.  The four methods launch one kernel each; the owner of
    the object reduces `pq`, `y`, `mass` and `out["out_tokens"]` over the ranks between them."""

    def __init__(self, p_shard, q_shard, v0: int, V_total: int, rank: int, world: int, tokens, mask: TreeMask,
                 gamma, u_accept, u_bonus):
        B, N, Vs = p_shard.shape
        _dev_tensor(p_shard, torch.float32, "p_shard")
        _dev_tensor(q_shard, torch.float32, "q_shard")
        _dev_tensor(tokens, torch.int32, "tokens")
        _dev_tensor(u_accept, torch.float32, "u_accept")
        _dev_tensor(u_bonus, torch.float32, "u_bonus")
        if gamma is not None:
            _dev_tensor(gamma, torch.int32, "gamma")
        if mask.n_nodes != N or tuple(q_shard.shape) != (B, N, Vs) or tuple(tokens.shape) != (B, N):
            raise ValueError("shape mismatch between p_shard, q_shard, tokens and the tree")
        dev = p_shard.device
        self.p, self.q, self.v0, self.V_total, self.rank, self.world = p_shard, q_shard, int(v0), int(V_total), rank, world
        self.tokens, self.mask, self.gamma, self.u_accept, self.u_bonus = tokens, mask, gamma, u_accept, u_bonus
        self.B, self.N, self.Vs = B, N, Vs
        nl = mask.n_levels
        self.pq = torch.zeros((B, N, 2), dtype=torch.float64, device=dev)
        self.y = torch.zeros((B, N), dtype=torch.float64, device=dev)
        self.mass = torch.zeros((world, B, 2), dtype=torch.float64, device=dev)
        self.workspace = new_workspace(mcsd_verify_shard_workspace_bytes(B, N), dev)
        self.out = {
            "accept_len": torch.empty(B, dtype=torch.int32, device=dev),
            "out_tokens": torch.empty((B, nl + 1), dtype=torch.int32, device=dev),
            "out_nodes": torch.empty((B, nl), dtype=torch.int32, device=dev),
            "best_root": torch.empty(B, dtype=torch.int32, device=dev),
            "next_roots": None,
        }

    def gather(self):
        m = self.mask
        with torch.cuda.device(self.p.device):
            st = lib.mcsd_verify_shard_gather(_ptr(self.p), _ptr(self.q), _ptr(self.tokens), _ptr(m.parent),
                                              _ptr(m.level_start), m.n_levels, _ptr(self.gamma), self.B, self.N,
                                              self.Vs, self.v0, self.V_total, _ptr(self.pq), _stream())
        _check(st, "mcsd_verify_shard_gather")

    def round(self, r: int):
        m = self.mask
        with torch.cuda.device(self.p.device):
            st = lib.mcsd_verify_shard_round(_ptr(self.p), _ptr(self.q), _ptr(m.parent), _ptr(m.level_start),
                                             m.n_levels, _ptr(self.gamma), _ptr(self.u_accept), _ptr(self.pq),
                                             _ptr(self.y), r, self.B, self.N, self.Vs, _ptr(self.workspace),
                                             self.workspace.numel(), _stream())
        _check(st, "mcsd_verify_shard_round")

    def select(self):
        m, o = self.mask, self.out
        with torch.cuda.device(self.p.device):
            st = lib.mcsd_verify_shard_select(_ptr(self.p), _ptr(self.q), _ptr(self.tokens), m.n_levels, m.n_roots,
                                              self.B, self.N, self.Vs, self.v0, self.V_total, self.rank, self.world,
                                              _ptr(o["accept_len"]), _ptr(o["out_tokens"]), _ptr(o["out_nodes"]),
                                              _ptr(o["best_root"]), _ptr(self.mass), _ptr(self.workspace),
                                              self.workspace.numel(), _stream())
        _check(st, "mcsd_verify_shard_select")

    def pick(self):
        m = self.mask
        with torch.cuda.device(self.p.device):
            st = lib.mcsd_verify_shard_pick(_ptr(self.p), _ptr(self.q), _ptr(self.u_bonus), m.n_levels, self.B,
                                            self.N, self.Vs, self.v0, self.V_total, self.rank, self.world,
                                            _ptr(self.mass), _ptr(self.out["out_tokens"]), _ptr(self.workspace),
                                            self.workspace.numel(), _stream())
        _check(st, "mcsd_verify_shard_pick")


def shard_batch(B: int, rank: int, world_size: int):
    """Sequences [lo, hi) of a batch of B that rank `rank` of `world_size` verifies.

    Sequences are independent in every step of the path, so ranks split the batch and exchange nothing."""
    if world_size < 1 or not (0 <= rank < world_size):
        raise ValueError("bad rank/world_size")
    base, rem = divmod(B, world_size)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)
