"""Multi-GPU plumbing of the benchmark: replicas only.

Every (sequence, layer, value head) is an independent recurrence (Eq. 7 acts on the key side only and heads never
mix), so the path has no exchange step and no collective on the data path.  With N ranks every rank runs its own
replica of the workload; the only communication is the timing reduction below (max over ranks) on the benchmark's
process group.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def reduce_max(x: float, device="cpu") -> float:
    """Max of a host scalar over all ranks (identity without an initialised process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(nodes_per_rank: int, ms_per_step_local: float, device="cpu"):
    """Whole-job throughput of N replicas: (units all ranks processed) / (slowest rank's time).

    Returns ``(value_per_second, ms_per_step_max)``.
    """
    world = dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1
    ms = reduce_max(ms_per_step_local, device)
    return nodes_per_rank * world / (ms * 1e-3), ms
