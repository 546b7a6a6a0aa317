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


def _free_port() -> int:
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return int(s.getsockname()[1])


def spawn_ranks(n: int, argv: Sequence[str]) -> int:
    """Start `python -m torch.distributed.run` with n ranks of the script in argv[0] on this node
    (rendezvous on 127.0.0.1, a free port) and return its exit code.  The ranks are independent
    replicas: the launcher only gives them RANK / LOCAL_RANK / WORLD_SIZE and a store for the
    barrier and the MAX over their times."""
    import subprocess
    import sys
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={int(n)}",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port())] + list(argv)
    return subprocess.call(cmd)


def selftest(rank: int, world: int, gpus: int) -> None:
    """What a benchmark rank does around its timed region, on the CPU with gloo: rendezvous, barrier,
    MAX over the ranks' times, SUM of their units; rank 0 prints one JSON line.  Used by the tests to
    check that `--gpus N` without a launcher really starts N ranks and aggregates them."""
    import json
    if world > 1:
        dist.init_process_group("gloo")
    try:
        if world > 1:
            dist.barrier()
        ms = 10.0 * (rank + 1)                  # rank r pretends to need 10 (r + 1) ms for 1000 units
        thr = job_throughput(1000.0, ms)        # every rank takes part in the SUM and the MAX
        slowest = max_over_ranks(ms)
        if rank == 0:
            print(json.dumps({"selftest": True, "n_gpus": world, "asked_gpus": gpus, "ms": slowest, "value": thr}), flush=True)
    finally:
        if world > 1:
            dist.destroy_process_group()
