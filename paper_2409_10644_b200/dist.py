"""Multi-GPU plumbing: one process per GPU, sequences sharded over ranks, no data-path collective.

Every step of tree verification is independent per sequence, so N GPUs verify N batch shards side by
side (weak scaling).  The only communication is the bookkeeping below: units add up, time is the
slowest rank's.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def aggregate(units_local: float, ms_local: float, device="cpu"):
    """(sum over ranks of units, max over ranks of milliseconds); identity without a process group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(units_local), float(ms_local)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(u.item()), float(t.item())


# --------------------------------------------------------------------------------------------------
# Vocabulary-sharded verify: the one place on the path with a real exchange step.  When the target's
# output layer is tensor-parallel, every rank holds a slice of the vocabulary of p and q; the accept /
# reject walk then needs a few numbers per node summed over the ranks (see mcsd.h), never a full row.
# --------------------------------------------------------------------------------------------------

def vocab_shard_range(V_total: int, rank: int, world_size: int, align: int = 4):
    """Token ids [v0, v1) held by `rank`: contiguous, in rank order, covering [0, V_total); every boundary
    but the last is a multiple of `align` ids so that a rank's rows keep 16-byte loads."""
    if world_size < 1 or not (0 <= rank < world_size) or V_total < 1 or align < 1:
        raise ValueError("bad rank/world_size/V_total")
    units = (V_total + align - 1) // align
    if units < world_size:
        raise ValueError("vocabulary of %d ids is too small for %d ranks at %d-id alignment" % (V_total, world_size, align))
    base, rem = divmod(units, world_size)
    lo = (rank * base + min(rank, rem)) * align
    hi = lo + (base + (1 if rank < rem else 0)) * align
    return min(lo, V_total), min(hi, V_total)


def max_children(parent) -> int:
    """Largest number of children of any node of a parent array (roots carry -1)."""
    import numpy as np
    parent = np.asarray(parent)
    kids = parent[parent >= 0]
    return int(np.bincount(kids).max()) if kids.size else 0


def _all_reduce_group(group):
    def reduce(tensors, op):
        for t in tensors:
            dist.all_reduce(t, op=dist.ReduceOp.SUM if op == "sum" else dist.ReduceOp.MAX, group=group)
    return reduce


def reduce_on_one_device(tensors, op):
    """Stand-in for the all-reduce when all ranks' shards sit on one GPU (tests, single-GPU profiling): the
    ranks' buffers are combined in rank order and every rank gets the result.  Nothing waits on anything:
    the ranks' kernels are ordinary launches of one stream, one after the other."""
    stacked = torch.stack(list(tensors))
    red = stacked.sum(0) if op == "sum" else stacked.amax(0)
    for t in tensors:
        t.copy_(red)


def drive_vocab_shards(shards, reduce, k: int):
    """Issues the launches of the vocabulary-sharded verify step for the given rank objects (one per process
    in a real job) with `reduce(tensors, "sum" | "max")` between them; k = max_children(parent)."""
    for s in shards:
        s.gather()
    reduce([s.pq for s in shards], "sum")
    for r in range(k + 1):
        for s in shards:
            s.round(r)
        if r < k:
            reduce([s.y for s in shards], "sum")
    for s in shards:
        s.select()
    reduce([s.mass for s in shards], "sum")
    for s in shards:
        s.pick()
    reduce([s.out["out_tokens"] for s in shards], "max")
    return [s.out for s in shards]


def verify_tree_vocab_sharded(p_shard, q_shard, v0, V_total, tokens, mask, gamma, u_accept, u_bonus, group=None):
    """This rank's part of a vocabulary-sharded verify step over the default (or given) process group; returns
    the same outputs as mcsd_verify_tree on every rank.  k + 3 small all-reduces (k = widest sibling group)."""
    from .binding import VocabShard
    rank = dist.get_rank(group) if dist.is_initialized() else 0
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    shard = VocabShard(p_shard, q_shard, v0, V_total, rank, world, tokens, mask, gamma, u_accept, u_bonus)
    k = max_children(mask.parent.cpu().numpy())
    reduce = _all_reduce_group(group) if world > 1 else (lambda tensors, op: None)
    return drive_vocab_shards([shard], reduce, k)[0]
