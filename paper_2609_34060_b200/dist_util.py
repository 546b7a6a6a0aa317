"""Multi-GPU bookkeeping for the benchmark: the path has no exchange step, so ranks are
independent replicas (or shards of a request list) and only the *timing* is combined.

Every (layer, head, token) of apply / chain / project is independent, so there is no
data-path collective; the only communication is a barrier around the timed region and a
MAX over the ranks' device times.
"""
from __future__ import annotations

from typing import List, Sequence

import torch
import torch.distributed as dist


def shard(units: Sequence, rank: int, world: int) -> List:
    """Contiguous, balanced shard of a list of independent units (requests) for one rank."""
    n = len(units)
    lo, hi = n * rank // world, n * (rank + 1) // world
    return list(units[lo:hi])


def max_over_ranks(value: float, device="cpu") -> float:
    """MAX of a per-rank scalar (device time in ms); identity without a process group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    """SUM of a per-rank scalar (units processed)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(units_local: float, ms_local: float, device="cpu") -> float:
    """Whole-job throughput: units all ranks processed divided by the slowest rank's time."""
    total = sum_over_ranks(units_local, device)
    ms = max_over_ranks(ms_local, device)
    return total / (ms * 1e-3)
