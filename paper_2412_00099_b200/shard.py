"""Multi-GPU layout: replicas only.

Token streams are independent (each has its own cache state, Delta statistics and counters), so the
workload shards by giving every rank its own set of streams and a full copy of the weights.  The data
path has no exchange step; the only cross-rank operations are the timing maximum and the sum of the
miss counters, both on a handful of scalars.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def replica_seed(seed: int, rank: int) -> int:
    """Seed of the streams owned by `rank`: rank 0 reproduces the single-GPU workload."""
    return seed + 1000 * rank


def stream_range(n_streams_total: int, rank: int, world: int):
    """Contiguous block of a global stream set owned by `rank` (sizes differ by at most one)."""
    lo = n_streams_total * rank // world
    hi = n_streams_total * (rank + 1) // world
    return lo, hi


def _reduce(value, device, op):
    if device is None or not dist.is_initialized():
        return value
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=op)
    return t.item()


def reduce_max(value: float, device) -> float:
    return _reduce(float(value), device, dist.ReduceOp.MAX)


def reduce_sum(value: float, device) -> float:
    return _reduce(float(value), device, dist.ReduceOp.SUM)
