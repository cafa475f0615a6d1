"""Replica bookkeeping for multi-GPU runs.

The path has no exchange step: requests are independent, so N GPUs run N independent
replicas of the workload (one process per GPU) and only the timing is combined:
the job's time is the slowest rank's, the job's work is the sum over ranks.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def replica_streams(rank: int, n_per_rank: int) -> list:
    """Seed-stream ids of the request replicas a rank generates (disjoint across ranks)."""
    return [100 + rank * n_per_rank + r for r in range(n_per_rank)]


def combine(units_local: float, ms_local: float, device="cpu"):
    """(sum of units over ranks, max of elapsed ms over ranks).  Without an initialised
    process group the local values are returned."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(units_local), float(ms_local)
    u = torch.tensor([float(units_local)], dtype=torch.float64, device=device)
    t = torch.tensor([float(ms_local)], dtype=torch.float64, device=device)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(u.item()), float(t.item())


def throughput(units_local: float, ms_local: float, device="cpu") -> float:
    """Whole-job units per second."""
    units, ms = combine(units_local, ms_local, device)
    return units / (ms * 1e-3)
