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
