#!/usr/bin/env python
"""Benchmark of the KV-correction hot path on B200.

One *step* is one pass of the whole path over one synthetic request of the named
workload: for every workflow edge a -> a+1 the rank-r state is built from the pair of
true caches (kvc_state_update, FIT mode: deviation, Gram, eigensolve, projection), then
the corrected caches of agents 1..N-1 are materialised from agent 0's exact cache
(kvc_chain).  `value` is the algorithmic HBM bytes of those launches divided by the
device time of the step (CUDA events), inputs resident in HBM; `e2e` is the same with
the step's inputs copied from pinned host memory and the corrected caches copied back
inside the timed region.  `roofline` is for the dominant kernel (one hop of the apply
stream) against the measured HBM copy bandwidth of this machine.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

With --impl reference the fp64 CPU oracle is timed instead, on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2609_34060_b200 import dist_util  # noqa: E402
from paper_2609_34060_b200 import workloads as wl  # noqa: E402

METRIC = "corrected-KV GB/s (algorithmic HBM bytes / time), whole hot path"
UNIT = "GB/s"
HBM_FALLBACK_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of one apply launch on the 8K workload, from the ncu
# capture summarised in profiles/apply_tc_kernel_dram_traffic_L16.md: measured at L = 16
# (811.95 MB read + 493.36 MB written per launch) and scaled by 2 to L = 32 (traffic is
# proportional to the token-slabs processed).  None for other workloads.
APPLY_TRAFFIC_BYTES_LLAMA8B_8K = 2 * (811_950_000 + 493_360_000)


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return HBM_FALLBACK_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                continue
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def _dist():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


# --------------------------------------------------------------------------------------
# the library arm
# --------------------------------------------------------------------------------------


def build_workload(cfg: wl.Config, dev, kvc, only="all", grouped=False):
    """Everything one step reads, resident on the device.  Draws come from the seeded
    generator; the true target caches are derived with the library itself (aligned
    source + exact rank-r deviation, then N(0, sigma) noise, rounded to bf16)."""
    rope = kvc.Rope(cfg.theta)
    pl = wl.prefix_lengths(cfg)
    n = cfg.n_agents
    if cfg.paged:
        npg = wl.n_pages(cfg.T, cfg.page)
        P = npg + 8
        tables = [wl.page_table(npg, P, cfg.seed, a, dev) for a in range(2 * n)]
        k0, v0 = wl.base_cache(cfg, dev, table=tables[0], n_phys=P)
        mk = lambda t: kvc.Cache(torch.empty_like(k0), torch.empty_like(v0), T=cfg.T, page_table=t)
        a0 = kvc.Cache(k0, v0, T=cfg.T, page_table=tables[0])
    else:
        k0, v0 = wl.base_cache(cfg, dev)
        mk = lambda t: kvc.Cache(torch.empty_like(k0), torch.empty_like(v0))
        tables = [None] * (2 * n)
        a0 = kvc.Cache(k0, v0)
    true = [a0]
    if only in ("apply", "gate", "multi", "weights"):
        # the chain (or the gate) alone: the generator's states are used directly, no targets needed
        states = []
        for a in range(1, n):
            if grouped:     # one state per layer over all KV heads (D = H d): coeff [L,T,r], basis [L,r,H d]
                mkc = lambda tag: wl.coefficients(cfg.L, 1, cfg.T, cfg.r, cfg.seed, 4 * a + tag, dev)[:, 0].contiguous()
                mkb = lambda tag: wl.orthonormal_basis(cfg.L, 1, cfg.r, cfg.H * cfg.d, cfg.seed, 4 * a + tag, dev)[:, 0].contiguous()
                states.append(kvc.State(mkc(0), mkc(1), mkb(2), mkb(3), grouping=kvc.KVC_GROUP_LAYER))
                continue
            s = wl.hop_state(cfg, a, dev)
            states.append(kvc.State(s["coeff_k"], s["coeff_v"], s["basis_k"], s["basis_v"]))
        if only == "gate":
            # the reliability gate over a pool whose anchors are the hop states' value factors
            f64 = lambda m: torch.empty(m, dtype=torch.float64, device=dev)
            return {"rope": rope, "pl": pl, "true": true, "states": states, "outs": [], "ws": None, "only": only,
                    "gate": (f64(n - 1), f64(n - 1), f64(1))}
        if only == "weights":
            # App. A.3 token-wise weights: the hop states act as the base factorisations of n - 1 anchors
            tp = kvc.kvc_multi_tpad(cfg.T)
            w = [torch.empty(n - 1, tp, device=dev) for _ in range(2)]
            ws = torch.empty(kvc.kvc_token_weights_workspace_bytes(a0, n - 1), dtype=torch.uint8, device=dev)
            return {"rope": rope, "pl": pl, "true": true, "states": states, "outs": [], "ws": ws, "only": only, "w": w}
        if only == "multi":
            # Eq. 8: the hop states act as the corrections stored in n - 1 anchors, with seeded token-wise weights
            tp = kvc.kvc_multi_tpad(cfg.T)
            g = torch.Generator(device=dev)
            g.manual_seed(cfg.seed * 7919 + 99)
            w = [torch.rand(n - 1, tp, device=dev, generator=g) + 0.05 for _ in range(2)]
            w = [(x / x.sum(dim=0, keepdim=True)).contiguous() for x in w]
            ws = torch.empty(kvc.kvc_multi_workspace_bytes(a0, states), dtype=torch.uint8, device=dev)
            return {"rope": rope, "pl": pl, "true": true, "states": states, "outs": [mk(tables[n + 1])], "ws": ws,
                    "only": only, "w": w}
        outs = [mk(tables[n + a]) for a in range(1, n)]
        return {"rope": rope, "pl": pl, "true": true, "states": states, "outs": outs, "ws": None, "only": only}
    for a in range(1, n):
        s = wl.hop_state(cfg, a, dev)
        st = kvc.State(s["coeff_k"], s["coeff_v"], s["basis_k"], s["basis_v"])
        tgt = mk(tables[a])
        kvc.kvc_apply(true[-1], st, pl[a] - pl[a - 1], rope, tgt)
        for t, tag in ((tgt.k, 0), (tgt.v, 1)):      # noise below one bf16 step mostly dithers the rounding
            flat = t.view(-1)
            chunk = 1 << 26
            g = torch.Generator(device=dev)
            g.manual_seed(cfg.seed * 7919 + 2 * a + tag)
            for o in range(0, flat.numel(), chunk):
                seg = flat[o:o + chunk]
                seg.copy_((seg.float() + cfg.sigma * torch.randn(seg.numel(), device=dev, generator=g)).to(torch.bfloat16))
        true.append(tgt)
        del s, st
    torch.cuda.synchronize()
    L, H, T, d, r = cfg.L, cfg.H, cfg.T, cfg.d, cfg.r
    states = [kvc.State(torch.empty(L, H, T, r, device=dev), torch.empty(L, H, T, r, device=dev),
                        torch.empty(L, H, r, d, device=dev), torch.empty(L, H, r, d, device=dev)) for _ in range(n - 1)]
    outs = [mk(tables[n + a]) for a in range(1, n)]
    ws = torch.empty(max(kvc.kvc_chain_update_workspace_bytes(true, states, kvc.KVC_FIT_FAST), 256), dtype=torch.uint8, device=dev)
    return {"rope": rope, "pl": pl, "true": true, "states": states, "outs": outs, "ws": ws, "only": only}


def build_ring(cfg: wl.Config, dev, kvc):
    """Long-context chain that does not fit with every agent's cache resident (config 5): agent 0's
    cache, two output buffers used in turn, one coefficient set shared by all hops (the shift still
    differs per hop).  Apply only: there are no resident true targets to fit states from."""
    rope = kvc.Rope(cfg.theta)
    pl = wl.prefix_lengths(cfg)
    npg = wl.n_pages(cfg.T, cfg.page)
    P = npg + 8
    tables = [wl.page_table(npg, P, cfg.seed, a, dev) for a in range(3)]
    k0, v0 = wl.base_cache(cfg, dev, table=tables[0], n_phys=P)
    a0 = kvc.Cache(k0, v0, T=cfg.T, page_table=tables[0])
    ring = [kvc.Cache(torch.empty_like(k0), torch.empty_like(v0), T=cfg.T, page_table=tables[1 + i]) for i in range(2)]
    s = wl.hop_state(cfg, 1, dev)
    st = kvc.State(s["coeff_k"], s["coeff_v"], s["basis_k"], s["basis_v"])
    return {"kind": "ring", "rope": rope, "pl": pl, "a0": a0, "ring": ring, "st": st, "true": [a0], "states": [st] * (cfg.n_agents - 1),
            "only": "apply"}


def build_serving(n_requests: int, dev, kvc, seed=0, L=32, H=8, d=128, page=16, theta=500000.0):
    """Config 4: a ragged serving batch.  One shared page pool holds two copies of every request's
    cache (source and destination of a hop round alternate); hop round h is ONE kvc_apply_batch
    over all requests that have more than h agents."""
    reqs = wl.serving_batch(n_requests, seed=seed)
    rope = kvc.Rope(theta)
    pages = [wl.n_pages(r.T, page) for r in reqs]
    P = 2 * sum(pages) + 16
    perm = wl.page_table(P, P, seed, 900, "cpu")
    pool_k = torch.empty((L, P, H, page, d), dtype=torch.bfloat16, device=dev)
    pool_v = torch.empty((L, P, H, page, d), dtype=torch.bfloat16, device=dev)
    g = torch.Generator(device=dev)
    g.manual_seed(seed * 7919 + 4)
    for t in (pool_k, pool_v):
        for l in range(L):
            t[l].normal_(generator=g)
    caches, states, off = [], [], 0
    for i, r in enumerate(reqs):
        ta = perm[off: off + pages[i]].contiguous().to(dev)
        tb = perm[off + pages[i]: off + 2 * pages[i]].contiguous().to(dev)
        off += 2 * pages[i]
        caches.append((kvc.Cache(pool_k, pool_v, T=r.T, page_table=ta), kvc.Cache(pool_k, pool_v, T=r.T, page_table=tb)))
        c = wl.Config(f"rq{i}", L=L, H=H, d=d, T=r.T, n_agents=r.n_agents, r=r.r, theta=theta, seed=seed * 1000 + i)
        s = wl.hop_state(c, 1, dev)
        states.append(kvc.State(s["coeff_k"], s["coeff_v"], s["basis_k"], s["basis_v"]))
    rounds = []
    for h in range(1, max(r.n_agents for r in reqs)):
        items = [kvc.Item(caches[i][(h - 1) % 2], caches[i][h % 2], states[i], r.prefix[h] - r.prefix[h - 1])
                 for i, r in enumerate(reqs) if r.n_agents > h]
        rounds.append(items)
    # a round runs as one kernel per rank class present (r <= 32, r > 32)
    kernels = sum(len({r.r <= 32 for r in reqs if r.n_agents > h}) for h in range(1, max(r.n_agents for r in reqs)))
    nb = kvc.kvc_batch_workspace_bytes(n_requests)
    ws = [torch.empty(nb, dtype=torch.uint8, device=dev) for _ in rounds]
    staging = [torch.empty(nb, dtype=torch.uint8).pin_memory() for _ in rounds]
    app = sum(kvc.kvc_apply_bytes(it.src, it.st) for items in rounds for it in items)
    return {"kind": "serving", "rope": rope, "rounds": rounds, "ws": ws, "staging": staging, "reqs": reqs, "apply_bytes": app,
            "only": "apply", "launches": len(rounds), "kernels": kernels, "tokens": sum(r.T for r in reqs)}


def run_step(W, kvc, ev=None):
    """One pass of the path.  `ev` (optional) collects CUDA-event pairs per kernel family."""
    pl, rope, n = W.get("pl"), W["rope"], len(W.get("true", []))

    def mark(name):
        if ev is None:
            return None
        e = torch.cuda.Event(enable_timing=True)
        e.record()
        ev.setdefault(name, []).append(e)
        return e

    only = W.get("only", "all")
    if W.get("kind") == "ring":
        mark("chain_begin")
        cur = W["a0"]
        for a in range(1, len(pl)):
            dst = W["ring"][a % 2]
            kvc.kvc_apply(cur, W["st"], pl[a] - pl[a - 1], rope, dst)
            cur = dst
        mark("chain_end")
        return
    if W.get("kind") == "serving":
        mark("chain_begin")
        for items, ws, stg in zip(W["rounds"], W["ws"], W["staging"]):
            kvc.kvc_apply_batch(items, rope, ws, stg)
        mark("chain_end")
        return
    if only == "gate":
        d2, g, ent = W["gate"]
        mark("chain_begin")
        kvc.kvc_gate_distance(W["true"][0], W["states"], W["true"][0].T, d2)
        kvc.kvc_gate_weights(d2, g, ent)
        mark("chain_end")
        return
    if only == "weights":
        mark("chain_begin")
        kvc.kvc_token_weights(W["true"][0], pl[0], W["states"], pl[1:], rope, W["w"][0], W["w"][1], W["ws"])
        mark("chain_end")
        return
    if only == "multi":
        mark("chain_begin")
        kvc.kvc_apply_multi(W["true"][0], W["states"], W["w"][0], W["w"][1], pl[1] - pl[0], rope, W["outs"][0], W["ws"])
        mark("chain_end")
        return
    if only != "apply":
        mark("update_begin")
        if W.get("edges", "chain") == "chain":     # every edge's state in one call: one eigensolver launch for all
            kvc.kvc_state_update_chain(W["true"], pl, rope, W["states"], W.get("fit_mode", kvc.KVC_FIT_FAST),
                                       workspace=W["ws"])
        else:
            for a in range(1, n):
                kvc.kvc_state_update(W["true"][a - 1], W["true"][a], pl[a] - pl[a - 1], rope, W["states"][a - 1],
                                     W.get("fit_mode", kvc.KVC_FIT_FAST), workspace=W["ws"])
        mark("update_end")
    if only != "update":
        mark("chain_begin")
        if W.get("chain_ws") is not None:
            kvc.kvc_chain_fused(W["true"][0], pl, W["states"], rope, W["outs"], W["chain_ws"])
        else:
            kvc.kvc_chain(W["true"][0], pl, W["states"], rope, W["outs"])
        mark("chain_end")


def step_bytes(W, kvc):
    if W.get("kind") == "serving":
        return 0, W["apply_bytes"]
    n = len(W["states"]) + 1
    only = W.get("only", "all")
    if only == "gate":      # per anchor: the source's values (2d B per token-slab) + value coefficients (4r) + basis
        c = W["true"][0]
        return 0, sum(c.L * c.H * (c.T * (2 * c.d + 4 * s.r) + 4 * s.r * c.d) for s in W["states"])
    if only == "weights":   # per anchor: the source cache (4d B per token-slab) + key and value coefficients (8r) + bases
        c = W["true"][0]
        return 0, sum(c.L * c.H * (c.T * (4 * c.d + 8 * s.r) + 8 * s.r * c.d) for s in W["states"])
    if only == "multi":     # caches in and out (4d + 4d), every anchor's coefficients (8r) and weights (8 B per token)
        c = W["true"][0]
        return 0, c.L * c.H * c.T * (8 * c.d + sum(8 * s.r for s in W["states"])) + 8 * len(W["states"]) * c.T \
            + sum(8 * s.r * c.d * c.L * c.H for s in W["states"])
    upd = 0 if only == "apply" else sum(kvc.kvc_update_bytes(W["true"][0], W["states"][a - 1], kvc.KVC_FIT, True)
                                         for a in range(1, n))
    app = 0 if only == "update" else sum(kvc.kvc_apply_bytes(W["true"][0], W["states"][a - 1]) for a in range(1, n))
    return upd, app


def cpu_baseline(cfg: wl.Config, budget_s: float = 20.0):
    """The fp64 oracle, as it stands, on a bounded sample of the same workload: whole
    (layer, head) slabs -- all tokens, all hops: FIT update then chain -- until the
    time budget is used.  Returns the same metric (algorithmic bytes / wall time)."""
    import numpy as np
    from oracle import kvc_oracle as orc
    try:
        from threadpoolctl import threadpool_info
        cores = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    one = cfg.scaled(L=1, H=1, paged=False)
    pl = wl.prefix_lengths(cfg)
    f = orc.rope_inv_freq(cfg.d, cfg.theta)
    bits = lambda t: t.contiguous().view(torch.int16).numpy().view(np.uint16)
    done, t_used, nbytes = 0, 0.0, 0
    per_slab = None
    while done < cfg.L * cfg.H and (per_slab is None or t_used + per_slab <= budget_s):
        c = one.scaled(seed=cfg.seed + 1000 + done)
        k0, v0 = wl.base_cache(c, "cpu")
        true = [orc.Cache(bits(k0), bits(v0))]
        for a in range(1, cfg.n_agents):                       # untimed: derive the true targets
            s = wl.hop_state(c, a, "cpu")
            st = orc.State(*(s[x].numpy() for x in ("coeff_k", "coeff_v", "basis_k", "basis_v")))
            nk = wl.noise((1, 1, c.T, c.d), c.seed, 2 * a).numpy()
            nv = wl.noise((1, 1, c.T, c.d), c.seed, 2 * a + 1).numpy()
            true.append(orc.make_target(true[-1], st, pl[a] - pl[a - 1], f, nk, nv, c.sigma))
        t0 = time.perf_counter()
        states = []
        for a in range(1, cfg.n_agents):
            st, _ = orc.state_update(true[a - 1], true[a], pl[a] - pl[a - 1], f, r=cfg.r, mode=orc.FIT)
            states.append(st)
        orc.chain(true[0], pl, states, f)
        dt = time.perf_counter() - t0
        per_slab = dt if per_slab is None else max(per_slab, dt)
        t_used += dt
        done += 1
        hops = cfg.n_agents - 1
        tok = cfg.T
        apply_b = hops * (tok * (8 * cfg.d + 8 * cfg.r) + 2 * cfg.r * cfg.d * 4)
        upd_b = hops * (2 * tok * 8 * cfg.d + tok * 8 * cfg.r + 2 * cfg.r * cfg.d * 4 + 4 * cfg.d * cfg.d * 4)
        nbytes += apply_b + upd_b
    return {"value": nbytes / t_used / 1e9, "unit": UNIT, "cores": int(cores), "kind": "oracle",
            "sample": f"{done} of {cfg.L * cfg.H} (layer, head) slabs, all {cfg.T} tokens, all {cfg.n_agents - 1} hops "
                      f"(FIT update + chain), {t_used:.1f} s"}, t_used


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="llama8b_8k", choices=sorted(wl.CONFIGS) + ["serve64"])
    ap.add_argument("--requests", type=int, default=64, help="serve64: number of concurrent requests")
    ap.add_argument("--impl", default="kvc", choices=["kvc", "reference"])
    ap.add_argument("--path", default="auto", choices=["auto", "generic", "tc"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-budget", type=float, default=20.0)
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (small profiling cases)")
    ap.add_argument("--rank", type=int, default=0, help="override the rank r (experiments)")
    ap.add_argument("--chain", default="hops", choices=["hops", "fused"],
                    help="hops: kvc_chain, one launch per hop; fused: kvc_chain_fused, one pass over agent 0's cache")
    ap.add_argument("--fit", default="fast", choices=["fast", "full"],
                    help="fast: KVC_FIT_FAST (top-r subspace solver, full eigensolver where it declines); full: KVC_FIT")
    ap.add_argument("--edges", default="chain", choices=["chain", "each"],
                    help="chain: kvc_state_update_chain, all edges in one call; each: one kvc_state_update per edge")
    ap.add_argument("--grouped", type=int, default=0, help="1: per-layer states (D = H d), with --only apply")
    ap.add_argument("--paged", type=int, default=-1, help="override the layout: 1 paged, 0 contiguous (experiments)")
    ap.add_argument("--only", default="all", choices=["all", "apply", "update", "gate", "multi", "weights"],
                    help="profiling aid: time only the chain or only the state updates")
    args = ap.parse_args()
    rank, world, local = _dist()
    serving = args.workload == "serve64"
    cfg = wl.CONFIGS["llama8b_8k" if serving else args.workload]
    if args.layers > 0:
        cfg = cfg.scaled(L=args.layers)
    if args.rank > 0:
        cfg = cfg.scaled(r=args.rank)
    if args.paged >= 0:
        cfg = cfg.scaled(paged=bool(args.paged), image_spans=())
    ring = (not serving) and cfg.paged and cfg.n_agents * cfg.L * cfg.H * cfg.T * cfg.d * 8 > 100e9
    if serving or ring:
        args.only, args.no_e2e, args.no_cpu_baseline = "apply", True, True
    wname = (f"serve64: {args.requests} requests, L={cfg.L} Hkv={cfg.H} d={cfg.d}, T lognormal(median 4096) in [1k,32k], "
             f"3-6 agents, r in {{16,32,64}}, paged16, one ragged launch per hop round" if serving else
             f"{cfg.name}: L={cfg.L} Hkv={cfg.H} d={cfg.d} T={cfg.T} agents={cfg.n_agents} r={cfg.r} "
             f"{'paged16' if cfg.paged else 'contiguous'} bf16, seed {cfg.seed}" + (" (two output buffers in turn)" if ring else ""))
    config = {"workload": wname,
              "step": (f"kvc_state_update_chain({'FIT_FAST' if args.fit == 'fast' else 'FIT'}) over all edges"
                       if args.edges == "chain" else
                       f"per edge: kvc_state_update({'FIT_FAST' if args.fit == 'fast' else 'FIT'})") + " ; then kvc_chain over all agents",
              "l2": "inputs larger than L2 (126 MB): no flush between iterations", "parallelism": f"replicas x{world}",
              "only": args.only}

    if args.impl == "reference":
        if rank != 0:
            return
        steps = max(1, min(args.steps, 3))
        vals = []
        for _ in range(min(args.warmup, 1)):
            cpu_baseline(cfg, 3.0)
        t_all = 0.0
        for _ in range(steps):
            cb, t = cpu_baseline(cfg, max(2.0, 60.0 / steps))
            vals.append(cb["value"])
            t_all += t
        v = sum(vals) / len(vals)
        cb["value"] = v
        print(json.dumps({"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
                          "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": 1e3 * t_all / steps,
                          "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
                          "data": "synthetic", "config": config, "cpu_baseline": cb,
                          "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return

    import paper_2609_34060_b200 as kvc
    from paper_2609_34060_b200 import build as kbuild
    if not os.path.exists(kvc.LIB_PATH):
        kbuild.build()
    kvc.load()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    kvc.kvc_set_path({"auto": kvc.KVC_PATH_AUTO, "generic": kvc.KVC_PATH_GENERIC, "tc": kvc.KVC_PATH_TC}[args.path])

    if serving:
        W = build_serving(args.requests, dev, kvc, seed=rank, L=cfg.L)      # each rank serves its own batch
    elif ring:
        W = build_ring(cfg.scaled(seed=cfg.seed + rank), dev, kvc)
    else:
        W = build_workload(cfg.scaled(seed=cfg.seed + rank), dev, kvc, args.only, grouped=bool(args.grouped) and args.only == "apply")
    W["fit_mode"] = kvc.KVC_FIT_FAST if args.fit == "fast" else kvc.KVC_FIT
    W["edges"] = args.edges
    if args.chain == "fused" and W.get("kind") is None and W.get("outs") and args.only in ("all", "apply"):
        W["chain_ws"] = torch.empty(max(kvc.kvc_chain_workspace_bytes(W["true"][0], cfg.n_agents), 128), dtype=torch.uint8,
                                    device=dev)
    if args.only != "all":
        args.no_e2e = True
    upd_b, app_b = step_bytes(W, kvc)
    hops = W["launches"] if serving else (1 if args.only == "multi" else cfg.n_agents - 1)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        run_step(W, kvc)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ev = {}
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_begin.record()
    step_marks = []
    for _ in range(args.steps):
        run_step(W, kvc, ev)
        m = torch.cuda.Event(enable_timing=True)
        m.record()
        step_marks.append(m)
    t_end.record()
    barrier()
    per_step = [a.elapsed_time(b) for a, b in zip([t_begin] + step_marks[:-1], step_marks)]
    clocks = sampler.stop() if rank == 0 else None
    ms_total = t_begin.elapsed_time(t_end)
    chain_ms = sum(b.elapsed_time(e) for b, e in zip(ev.get("chain_begin", []), ev.get("chain_end", []))) / args.steps
    upd_ms = sum(b.elapsed_time(e) for b, e in zip(ev.get("update_begin", []), ev.get("update_end", []))) / args.steps
    chain_ms, upd_ms = max(chain_ms, 1e-9), max(upd_ms, 1e-9)
    last_path = kvc.kvc_last_path()
    flags = kvc.kvc_status_poll()
    assert flags == 0, f"a kernel flagged an anomaly: {flags}"
    ms_step = dist_util.max_over_ranks(ms_total, dev) / args.steps
    value = world * (upd_b + app_b) / (ms_step * 1e-3) / 1e9

    # end to end: inputs from pinned host memory, corrected caches back to the host
    e2e = None
    if not args.no_e2e:
        srcs = [c for c in W["true"]]
        host_in = [(c.k.cpu().pin_memory(), c.v.cpu().pin_memory()) for c in srcs]
        host_out = [(torch.empty_like(o.k, device="cpu").pin_memory(), torch.empty_like(o.v, device="cpu").pin_memory())
                    for o in W["outs"]]
        h2d = sum(k.numel() * 2 + v.numel() * 2 for k, v in host_in)
        d2h = sum(k.numel() * 2 + v.numel() * 2 for k, v in host_out)

        # Three streams: every step copies all its inputs in, runs the path and copies all its results
        # out; the copy-out of step i and the copy-in of step i + 1 share the link's two directions.
        # A step's kernels wait for its inputs and for the previous results to have left the device;
        # its copy-in waits for the previous step's kernels (they read the same buffers).
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        s_run = torch.cuda.current_stream()
        state = {"run_done": None, "out_done": None}

        def e2e_step():
            with torch.cuda.stream(s_in):
                if state["run_done"] is not None:
                    s_in.wait_event(state["run_done"])
                for c, (hk, hv) in zip(srcs, host_in):
                    c.k.copy_(hk, non_blocking=True)
                    c.v.copy_(hv, non_blocking=True)
                in_done = torch.cuda.Event()
                in_done.record(s_in)
            s_run.wait_event(in_done)
            if state["out_done"] is not None:
                s_run.wait_event(state["out_done"])
            run_step(W, kvc)
            state["run_done"] = torch.cuda.Event()
            state["run_done"].record(s_run)
            with torch.cuda.stream(s_out):
                s_out.wait_event(state["run_done"])
                for o, (hk, hv) in zip(W["outs"], host_out):
                    hk.copy_(o.k, non_blocking=True)
                    hv.copy_(o.v, non_blocking=True)
                state["out_done"] = torch.cuda.Event()
                state["out_done"].record(s_out)

        e2e_step()
        s_run.wait_event(state["out_done"])
        barrier()
        state["run_done"] = state["out_done"] = None
        n_e2e = max(1, min(args.steps, 5))
        b, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        b.record()
        s_in.wait_event(b)
        for _ in range(n_e2e):
            e2e_step()
        s_run.wait_event(state["out_done"])
        e.record()
        barrier()
        te = dist_util.max_over_ranks(b.elapsed_time(e), dev)
        e2e = {"value": world * (upd_b + app_b) / (te / n_e2e * 1e-3) / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": n_e2e}
        del host_in, host_out

    # beside the headline: the same chain through kvc_chain_fused (one pass over agent 0's cache, same bits)
    fused = None
    if rank == 0 and W.get("kind") is None and args.only in ("all", "apply") and W.get("chain_ws") is None and cfg.n_agents >= 3:
        cws = torch.empty(max(kvc.kvc_chain_workspace_bytes(W["true"][0], cfg.n_agents), 128), dtype=torch.uint8, device=dev)
        for _ in range(3):
            kvc.kvc_chain_fused(W["true"][0], W["pl"], W["states"], W["rope"], W["outs"], cws)
        fb, fe = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        fb.record()
        for _ in range(5):
            kvc.kvc_chain_fused(W["true"][0], W["pl"], W["states"], W["rope"], W["outs"], cws)
        fe.record()
        torch.cuda.synchronize()
        f_ms = fb.elapsed_time(fe) / 5
        c0 = W["true"][0]
        f_bytes = c0.L * c0.H * c0.T * (4 * c0.d + sum(8 * st.r + 4 * c0.d for st in W["states"]))
        fused = {"chain_ms": f_ms, "algorithmic_bytes": f_bytes, "GBs": f_bytes / (f_ms * 1e-3) / 1e9,
                 "us_per_agent_layer": f_ms * 1e3 / (cfg.n_agents - 1) / cfg.L}
        del cws
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peak, peak_kind = _peaks()
    hop_ms = chain_ms / hops
    # kernels of the state update per step: a Gram and a projection pass per edge, and the eigensolver
    # launches (FIT_FAST: subspace solver + full solver for what it declined), once for all edges or per edge
    eig_launches = (2 if args.fit == "fast" else 1) * (1 if args.edges == "chain" else hops)
    upd_launches = 2 * hops + eig_launches
    achieved = (app_b / hops) / (hop_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "gate distance (one anchor, Eq. 9)" if args.only == "gate" else "multi-anchor apply (Eq. 8)" if args.only == "multi" else "token-weight scores (one anchor, App. A.3)" if args.only == "weights" else "apply (one hop of kvc_chain)", "achieved": achieved, "peak": peak,
                "unit": "GB/s", "frac": achieved / peak, "peak_source": f"of {peak_kind}",
                "traffic": APPLY_TRAFFIC_BYTES_LLAMA8B_8K if (args.workload == "llama8b_8k" and args.layers == 0 and args.rank == 0 and args.paged < 0 and args.only not in ("gate", "multi", "weights") and not args.grouped) else None,
                "algorithmic_bytes_per_launch": app_b // hops,
                "us_per_launch": hop_ms * 1e3}
    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
           "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "bf16 storage, f32 accumulate", "data": "synthetic", "config": config,
           "clocks": clocks, "e2e": e2e,
           "gpu_launches": args.steps * W["kernels"] if serving else args.steps * (
               hops + 1 if args.only in ("gate", "multi", "weights") else
               (0 if args.only == "update" else hops) + (0 if args.only == "apply" else upd_launches)),
           "roofline": roofline,
           "breakdown": {"apply_GBs": achieved, "apply_frac_of_8TBs_nominal": achieved / 8000.0,
                         "us_per_agent_layer": hop_ms * 1e3 / cfg.L,
                         "output_only_GBs": (sum(o.nbytes() for o in W.get("outs", [])) / max(len(W.get("outs", [])), 1))
                         / (hop_ms * 1e-3) / 1e9 if W.get("outs") else None,
                         "step_ms_median": sorted(per_step)[len(per_step) // 2], "step_ms_min": min(per_step),
                         "update_fit_GBs": upd_b / (upd_ms * 1e-3) / 1e9, "update_ms_per_step": upd_ms,
                         "chain_ms_per_step": chain_ms, "chain_fused": fused,
                         "kernel_family": {0: "auto", 1: "generic (CUDA cores)", 2: "tc (TMA + tcgen05)"}[last_path]}}
    if not args.no_cpu_baseline:
        out["cpu_baseline"], _ = cpu_baseline(cfg, args.cpu_budget)
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
