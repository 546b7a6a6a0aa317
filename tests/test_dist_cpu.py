"""World-size-2 gloo test of the multi-rank bookkeeping bench.py uses (no GPU needed).

The hot path has no exchange step: ranks are replicas / shards, so what must be right is the
sharding of independent units and the way per-rank times are combined (MAX) with the units (SUM).
"""
import os

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_34060_b200 import dist_util
from paper_2609_34060_b200 import workloads as wl


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        reqs = wl.serving_batch(n_requests=11, seed=3)
        mine = dist_util.shard(reqs, rank, world)
        units = float(sum(r.T for r in mine))
        ms = 10.0 * (rank + 1)                      # rank 1 is the slow one
        dist.barrier()
        thr = dist_util.job_throughput(units, ms)
        q.put((rank, len(mine), units, dist_util.max_over_ranks(ms), thr))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_and_combine():
    world, port = 2, 29611
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    out = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    reqs = wl.serving_batch(n_requests=11, seed=3)
    total_tokens = float(sum(r.T for r in reqs))
    assert out[0][1] + out[1][1] == 11 and abs(out[0][1] - out[1][1]) <= 1      # balanced, nothing lost
    assert out[0][2] + out[1][2] == total_tokens
    for r in out:
        assert r[3] == 20.0                                                       # the slowest rank sets the time
        assert abs(r[4] - total_tokens / 20e-3) < 1e-6 * r[4]                     # whole-job units / max time


def test_single_process_is_identity():
    assert dist_util.max_over_ranks(3.5) == 3.5
    assert dist_util.job_throughput(100.0, 50.0) == 2000.0
    assert dist_util.shard(list(range(10)), 1, 3) == [3, 4, 5]


def test_bench_gpus_flag_starts_that_many_ranks():
    """`bench.py --gpus 2` outside a launcher starts two ranks itself; they rendezvous (gloo here),
    combine their times by MAX and their units by SUM, and exactly one JSON line comes out."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--selftest-dist"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = lines[0]
    assert rec["n_gpus"] == 2 and rec["asked_gpus"] == 2
    assert rec["ms"] == 20.0 and abs(rec["value"] - 2000.0 / 20e-3) < 1e-6 * rec["value"]
