"""Device-resident benchmark scenarios of the KV-correction hot path.

What `bench.py` times and what the full-size parity tests check are the same objects: a scenario is
everything one step of the path reads and writes, resident on the device, built from the seeded
generators of `workloads` (the true targets of the FIT updates are derived with the library's own
apply kernel from generator draws: aligned source + exact rank-r deviation + noise, rounded to bf16).
`run_step` issues one pass of the path over a scenario; `step_bytes` is its algorithmic HBM traffic.
"""
from __future__ import annotations

import torch

import paper_2609_34060_b200 as kvc
from . import workloads as wl

def build_workload(cfg: wl.Config, dev, only="all", grouped=False):
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

    def drawn_state(a):
        if grouped:     # one state per layer over all KV heads (D = H d): coeff [L,T,r], basis [L,r,H d]
            mkc = lambda tag: wl.coefficients(cfg.L, 1, cfg.T, cfg.r, cfg.seed, 4 * a + tag, dev)[:, 0].contiguous()
            mkb = lambda tag: wl.orthonormal_basis(cfg.L, 1, cfg.r, cfg.H * cfg.d, cfg.seed, 4 * a + tag, dev)[:, 0].contiguous()
            return kvc.State(mkc(0), mkc(1), mkb(2), mkb(3), grouping=kvc.KVC_GROUP_LAYER)
        s = wl.hop_state(cfg, a, dev)
        return kvc.State(s["coeff_k"], s["coeff_v"], s["basis_k"], s["basis_v"])

    if only in ("apply", "gate", "multi", "weights"):
        # the chain (or the gate) alone: the generator's states are used directly, no targets needed
        states = [drawn_state(a) for a in range(1, n)]
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
        st = drawn_state(a)
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
        del st
    torch.cuda.synchronize()
    L, H, T, d, r = cfg.L, cfg.H, cfg.T, cfg.d, cfg.r
    if grouped:
        states = [kvc.State(torch.empty(L, T, r, device=dev), torch.empty(L, T, r, device=dev),
                            torch.empty(L, r, H * d, device=dev), torch.empty(L, r, H * d, device=dev),
                            grouping=kvc.KVC_GROUP_LAYER) for _ in range(n - 1)]
    else:
        states = [kvc.State(torch.empty(L, H, T, r, device=dev), torch.empty(L, H, T, r, device=dev),
                            torch.empty(L, H, r, d, device=dev), torch.empty(L, H, r, d, device=dev)) for _ in range(n - 1)]
    outs = [mk(tables[n + a]) for a in range(1, n)]
    ws = torch.empty(max(kvc.kvc_chain_update_workspace_bytes(true, states, kvc.KVC_FIT_FAST), 256), dtype=torch.uint8, device=dev)
    return {"rope": rope, "pl": pl, "true": true, "states": states, "outs": outs, "ws": ws, "only": only}


def build_ring(cfg: wl.Config, dev, n_hops=None):
    """Long-context chain whose corrected caches are not all kept (config 5): agent 0's cache, two
    output buffers used in turn, and every hop's OWN state resident (distinct coefficients and bases
    per hop, drawn from the seeded generator).  At L=80, T=32768, r=64: 10.7 GB for agent 0, 21.5 GB for
    the two buffers, 10.7 GB per state.  Apply only: there are no resident true targets to fit from."""
    rope = kvc.Rope(cfg.theta)
    pl = wl.prefix_lengths(cfg)
    n_hops = cfg.n_agents - 1 if n_hops is None else n_hops
    pl = pl[: n_hops + 1]
    npg = wl.n_pages(cfg.T, cfg.page)
    P = npg + 8
    tables = [wl.page_table(npg, P, cfg.seed, a, dev) for a in range(3)]
    k0, v0 = wl.base_cache(cfg, dev, table=tables[0], n_phys=P)
    a0 = kvc.Cache(k0, v0, T=cfg.T, page_table=tables[0])
    ring = [kvc.Cache(torch.empty_like(k0), torch.empty_like(v0), T=cfg.T, page_table=tables[1 + i]) for i in range(2)]
    states = []
    for a in range(1, n_hops + 1):
        s = wl.hop_state(cfg, a, dev)
        states.append(kvc.State(s["coeff_k"], s["coeff_v"], s["basis_k"], s["basis_v"]))
    return {"kind": "ring", "rope": rope, "pl": pl, "a0": a0, "ring": ring, "true": [a0], "states": states, "only": "apply"}


def build_serving(n_requests: int, dev, seed=0, L=32, H=8, d=128, page=16, theta=500000.0):
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


def run_step(W, ev=None):
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
            kvc.kvc_apply(cur, W["states"][a - 1], pl[a] - pl[a - 1], rope, dst)
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


def step_bytes(W):
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
    if only == "update":
        app = 0
    elif W.get("chain_ws") is not None:
        # the fused chain reads agent 0's cache once (4d B per token-slab), every hop's coefficients (8r) and bases,
        # and writes every hop's cache (4d)
        c = W["true"][0]
        app = c.L * c.H * (c.T * (4 * c.d + sum(8 * s.r + 4 * c.d for s in W["states"])) + sum(8 * s.r * c.d for s in W["states"]))
    else:
        app = sum(kvc.kvc_apply_bytes(W["true"][0], W["states"][a - 1]) for a in range(1, n))
    return upd, app


