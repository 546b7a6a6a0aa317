"""KVC_FIT_FAST: the top-r subspace solver and its hand-over to the full eigensolver.

Every matrix of a KVC_FIT_FAST update is served by one of two solvers and the workspace says which
(kvc_fit_solver).  The tests drive both: a deviation of rank r over a noise floor (gap behind the r-th
eigenvalue: the subspace solver must take it), the same data at a rank below the signal rank, a flat
Gaussian cache and an all-zero cache (no gap: the full solver must take them), and a rank above 32
(never tried).  Whichever solver ran, the state is held to the same bar as KVC_FIT: the oracle's
eigenvalues, orthonormal rows, the oracle's projector where the spectrum is separated, the Eckart-Young
residual, coefficient columns that are orthogonal with the eigenvalues as energies.
"""
import numpy as np
import pytest
import torch

import paper_2609_34060_b200 as kvc
from paper_2609_34060_b200 import workloads as wl
from oracle import kvc_oracle as orc

import helpers as hp
from test_gpu_update import _edge

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

CFG_TINY = wl.CONFIGS["tiny"]
CFG_8B_S = wl.CONFIGS["llama8b_8k"].scaled(name="8b_small", L=2, H=2, T=700)
CFG_VLM_S = wl.CONFIGS["vlm_16k"].scaled(name="vlm_small", L=1, H=2, T=400, image_spans=())


@pytest.fixture(autouse=True)
def _clean_status():
    kvc.kvc_status_reset()
    yield
    assert kvc.kvc_status_poll() == 0


def _fit(src, tgt, shift, cfg, r, mode, n_cov=None):
    L, H, T, d = cfg.L, cfg.H, cfg.T, cfg.d
    n = T if n_cov is None else n_cov
    st = kvc.State(torch.zeros(L, H, n, r, device=DEV), torch.zeros(L, H, n, r, device=DEV),
                   torch.full((L, H, r, d), 3.0, device=DEV), torch.full((L, H, r, d), 3.0, device=DEV), n_cov=n)
    ws = torch.zeros(kvc.kvc_workspace_bytes(tgt, st, mode), dtype=torch.uint8, device=DEV)
    kvc.kvc_state_update(src, tgt, shift, kvc.Rope(cfg.theta), st, mode, workspace=ws)
    torch.cuda.synchronize()
    m = L * H * 2
    ev = ws.view(torch.float32)[2 * m * d * d: 2 * m * d * d + m * d].cpu().numpy().astype(np.float64).reshape(L, H, 2, d)
    return st, ws, ev


@pytest.mark.parametrize("cfg", [CFG_TINY, CFG_8B_S, CFG_VLM_S], ids=lambda c: c.name)
def test_gapped_spectrum_is_served_by_the_subspace_solver(cfg):
    src_cpu, tgt_cpu, osrc, otgt, true, shift = _edge(cfg)
    f = hp.inv_freq(cfg)
    ost, oev = orc.state_update(osrc, otgt, shift, f, r=cfg.r, mode=orc.FIT)
    src, tgt = hp.to_dev(src_cpu, DEV), hp.to_dev(tgt_cpu, DEV)
    r, d = cfg.r, cfg.d
    st, ws, ev = _fit(src, tgt, shift, cfg, r, kvc.KVC_FIT_FAST)
    solver = kvc.kvc_fit_solver(tgt, ws).cpu().numpy()
    assert np.all(solver == kvc.KVC_SOLVER_SUBSPACE), solver
    for l in range(cfg.L):
        for h in range(cfg.H):
            for i, (which, B_t, c_t, B_o) in enumerate((("k", st.basis_k, st.coeff_k, ost.basis_k),
                                                        ("v", st.basis_v, st.coeff_v, ost.basis_v))):
                dl = orc.deviation(osrc.get_bits(which, l, h), otgt.get_bits(which, l, h), shift, f, which == "k")
                w = oev[l, h, i]
                # the r leading eigenvalues; the others are reported as their mean: exact trace
                assert np.max(np.abs(ev[l, h, i, :r] - w[:r])) <= 1e-4 * w[0]
                assert np.allclose(ev[l, h, i, r:], ev[l, h, i, r]) and ev[l, h, i, r] <= ev[l, h, i, r - 1]
                assert abs(np.sum(ev[l, h, i]) - np.sum(w)) <= 1e-4 * np.sum(w)
                B = B_t[l, h].cpu().numpy().astype(np.float64)
                c = c_t[l, h].cpu().numpy().astype(np.float64)
                assert np.max(np.abs(B @ B.T - np.eye(r))) <= 1e-5
                assert np.all(B[np.arange(r), np.argmax(np.abs(B), axis=1)] > 0)
                Bo = B_o[l, h].astype(np.float64)
                assert np.linalg.norm(B.T @ B - Bo.T @ Bo) <= 1e-2
                tail = float(np.sum(w[r:]))
                res = float(np.sum((dl - c @ B) ** 2))
                assert res <= 1.001 * tail + 1e-6 * float(np.sum(w)), (res, tail)
                Gc = c.T @ c
                assert np.max(np.abs(Gc - np.diag(np.diag(Gc)))) <= 2e-3 * w[0]
                assert np.max(np.abs(np.diag(Gc) - w[:r])) <= 1e-3 * w[0]                  # in order, too
                # every row is an eigenvector of the oracle's Gram matrix to float32 level
                G = orc.gram(dl)
                assert np.max(np.linalg.norm(G @ B.T - B.T * np.diag(B @ G @ B.T)[None, :], axis=0)) <= 1e-4 * w[0]
    # the same call in KVC_FIT mode gives the same subspace
    st2, _, ev2 = _fit(src, tgt, shift, cfg, r, kvc.KVC_FIT)
    for B1, B2 in ((st.basis_k, st2.basis_k), (st.basis_v, st2.basis_v)):
        P1 = torch.einsum("lhrd,lhre->lhde", B1, B1)
        P2 = torch.einsum("lhrd,lhre->lhde", B2, B2)
        assert float((P1 - P2).abs().max()) <= 1e-3
    assert np.max(np.abs(ev[..., :r] - ev2[..., :r])) <= 1e-4 * np.max(ev2)
    # and the effective rank (at most r here) is the same from both sets of eigenvalues
    er = kvc.kvc_effective_rank(tgt, ws).cpu().numpy()
    for l in range(cfg.L):
        for h in range(cfg.H):
            for i in range(2):
                assert er[l, h, i] == orc.effective_rank(oev[l, h, i]) <= r


def test_no_gap_goes_to_the_full_solver():
    """Ranks below the signal rank, a flat Gaussian cache, zeros, and a rank beyond the subspace
    solver's limit: each matrix names the full solver, and the results meet KVC_FIT's checks."""
    cfg = CFG_8B_S.scaled(L=1, H=2, T=300, r=8)
    src_cpu, tgt_cpu, osrc, otgt, true, shift = _edge(cfg)
    f = hp.inv_freq(cfg)
    src, tgt = hp.to_dev(src_cpu, DEV), hp.to_dev(tgt_cpu, DEV)
    _, oev = orc.state_update(osrc, otgt, shift, f, r=8, mode=orc.FIT)
    d = cfg.d
    for r, want in ((4, "full"), (8, "subspace"), (12, "full"), (32, "full"), (40, "rank")):
        st, ws, ev = _fit(src, tgt, shift, cfg, r, kvc.KVC_FIT_FAST)
        solver = kvc.kvc_fit_solver(tgt, ws).cpu().numpy()
        if want == "subspace":
            assert np.all(solver == kvc.KVC_SOLVER_SUBSPACE), (r, solver)
        elif want == "rank":
            assert np.all(solver == kvc.KVC_SOLVER_FULL_RANK), (r, solver)
        else:
            assert np.all(solver > 0), (r, solver)
        for h in range(cfg.H):
            for i, (which, B_t, c_t) in enumerate((("k", st.basis_k, st.coeff_k), ("v", st.basis_v, st.coeff_v))):
                dl = orc.deviation(osrc.get_bits(which, 0, h), otgt.get_bits(which, 0, h), shift, f, which == "k")
                w = oev[0, h, i]
                if want != "subspace":
                    assert np.max(np.abs(ev[0, h, i] - w)) <= 1e-4 * w[0], r
                B = B_t[0, h].cpu().numpy().astype(np.float64)
                c = c_t[0, h].cpu().numpy().astype(np.float64)
                assert np.max(np.abs(B @ B.T - np.eye(r))) <= 1e-4, r
                res = float(np.sum((dl - c @ B) ** 2))
                assert res <= float(np.sum(w[r:])) + 8 * r * 1.2e-6 * w[0] + 1e-9 * float(np.sum(w)), r
    # a flat spectrum: the Gaussian cache factorised by itself
    st, ws, ev = _fit(None, src, 0, cfg, 8, kvc.KVC_FIT_FAST)
    solver = kvc.kvc_fit_solver(src, ws).cpu().numpy()
    assert np.all(solver[:, :, 1] > 0), solver           # values: no structure at all
    v = orc.bf16_to_f64(osrc.get_bits("v", 0, 1))
    w = np.linalg.eigvalsh(v.T @ v)[::-1]
    assert np.max(np.abs(ev[0, 1, 1] - w)) <= 1e-4 * w[0]
    # all zeros
    z = kvc.Cache(torch.zeros_like(src.k), torch.zeros_like(src.v))
    st, ws, ev = _fit(None, z, 0, cfg, 8, kvc.KVC_FIT_FAST)
    assert np.all(kvc.kvc_fit_solver(z, ws).cpu().numpy() == kvc.KVC_SOLVER_FULL_DEPENDENT)
    assert np.all(ev == 0) and torch.all(st.basis_k == 0) and torch.all(st.coeff_v == 0)


@pytest.mark.parametrize("d", [64, 128])
def test_clustered_spectra_either_solver(d):
    """The drawn clustered spectra of the KVC_FIT tests through KVC_FIT_FAST at ranks up to 32: whichever
    solver a matrix gets, orthonormal rows at rounding level and a residual at the tail energy; where
    the subspace solver served it, the r leading eigenvalues are the library's."""
    T = 512
    served = {0: 0, 1: 0}
    for trial in range(20):
        x, _ = wl.clustered_rows(T, d, seed=11, tag=100 * d + trial)
        xn = x.to(torch.float64).numpy()
        w = np.linalg.eigvalsh(xn.T @ xn)[::-1]
        g = torch.Generator().manual_seed(77 * d + trial)
        r = int(torch.randint(1, 33, (1,), generator=g))
        cache = kvc.Cache(x.reshape(1, 1, T, d).contiguous().to(DEV), x.reshape(1, 1, T, d).contiguous().to(DEV))
        cfg = wl.Config("cl", L=1, H=1, d=d, T=T, n_agents=2, r=r, theta=10000.0)
        st, ws, ev = _fit(None, cache, 0, cfg, r, kvc.KVC_FIT_FAST)
        assert kvc.kvc_status_poll() == 0, (trial, r)
        sv = int(kvc.kvc_fit_solver(cache, ws)[0, 0, 1])
        served[int(sv != 0)] += 1
        k_top = r if sv == 0 else d
        assert np.max(np.abs(ev[0, 0, 1, :k_top] - w[:k_top])) <= 1e-4 * w[0], (trial, r, sv)
        B = st.basis_v[0, 0].cpu().numpy().astype(np.float64)
        c = st.coeff_v[0, 0].cpu().numpy().astype(np.float64)
        live = np.abs(B).sum(axis=1) > 0
        k = int(live.sum())
        assert np.all(live[:k]) and k >= min(r, int(np.sum(w > 1e-5 * w[0]))), (trial, r, k)
        assert np.max(np.abs(B[:k] @ B[:k].T - np.eye(k))) <= 1e-5, (trial, r, sv)
        res = float(np.sum((xn - c @ B) ** 2))
        assert res <= float(np.sum(w[k:])) + 8 * r * 1.2e-6 * w[0] + 1e-9 * float(np.sum(w)), (trial, r, sv)
    print("clustered spectra served by subspace / full solver:", served)


def _chain_caches(cfg, n_agents):
    """n_agents caches on the device: agent 0 drawn, agent a = bf16(Align(agent a-1) + A_a B_a + noise),
    built by the oracle from generator draws (so every edge is a rank-r deviation over a noise floor)."""
    cfg = cfg.scaled(n_agents=n_agents)
    pl = wl.prefix_lengths(cfg)
    f = hp.inv_freq(cfg)
    cpu = hp.make_cache(cfg)
    o = hp.oracle_cache(cpu)
    caches = [hp.to_dev(cpu, DEV)]
    as_t = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
    for a in range(1, n_agents):
        nk = wl.noise((cfg.L, cfg.H, cfg.T, cfg.d), cfg.seed, 2 * a).numpy()
        nv = wl.noise((cfg.L, cfg.H, cfg.T, cfg.d), cfg.seed, 2 * a + 1).numpy()
        o = orc.make_target(o, hp.oracle_state(hp.make_state(cfg, a)), pl[a] - pl[a - 1], f, nk, nv, cfg.sigma)
        caches.append(hp.to_dev(kvc.Cache(as_t(o.k), as_t(o.v)), DEV))
    return caches, pl


@pytest.mark.parametrize("mode", ["fit_fast", "fit", "project"])
def test_chain_update_equals_edge_by_edge(mode):
    """kvc_state_update_chain (all eigensolves of a workflow in one launch) against one kvc_state_update
    per edge: the same kernels on the same data, so bases, coefficients, eigenvalues and solver codes
    agree bit for bit.  The per-edge results are themselves oracle-checked by the tests above."""
    kmode = {"fit_fast": kvc.KVC_FIT_FAST, "fit": kvc.KVC_FIT, "project": kvc.KVC_PROJECT}[mode]
    cfg = CFG_8B_S.scaled(L=2, H=3, T=333, r=16)
    n = 4
    caches, pl = _chain_caches(cfg, n)
    rope = kvc.Rope(cfg.theta)
    L, H, T, d, r = cfg.L, cfg.H, cfg.T, cfg.d, cfg.r

    def fresh():
        g = torch.Generator(device=DEV).manual_seed(5)
        B = torch.linalg.qr(torch.randn(L, H, d, r, device=DEV, generator=g))[0].transpose(-1, -2).contiguous()
        return kvc.State(torch.zeros(L, H, T, r, device=DEV), torch.zeros(L, H, T, r, device=DEV), B.clone(), B.clone())

    one = [fresh() for _ in range(n - 1)]
    ws1 = []
    for e in range(n - 1):
        ws = torch.zeros(max(kvc.kvc_workspace_bytes(caches[e + 1], one[e], kmode), 256), dtype=torch.uint8, device=DEV)
        kvc.kvc_state_update(caches[e], caches[e + 1], pl[e + 1] - pl[e], rope, one[e], kmode, workspace=ws)
        ws1.append(ws)
    allst = [fresh() for _ in range(n - 1)]
    total = kvc.kvc_chain_update_workspace_bytes(caches, allst, kmode)
    stride = kvc.kvc_chain_update_edge_stride(caches[1], allst[0], kmode)
    assert total == (n - 1) * stride and stride % 256 == 0
    wsn = torch.zeros(max(total, 256), dtype=torch.uint8, device=DEV)
    kvc.kvc_state_update_chain(caches, pl, rope, allst, kmode, workspace=wsn)
    torch.cuda.synchronize()
    for e in range(n - 1):
        for name in ("coeff_k", "coeff_v", "basis_k", "basis_v"):
            assert torch.equal(getattr(one[e], name), getattr(allst[e], name)), (e, name)
        if kmode != kvc.KVC_PROJECT:
            sub = wsn[e * stride:(e + 1) * stride]
            m = L * H * 2
            lo, hi = 2 * m * d * d * 4, 2 * m * d * d * 4 + m * d * 4
            assert torch.equal(sub[lo:hi], ws1[e][lo:hi])                       # eigenvalues
            assert torch.equal(sub[:m * d * d * 4], ws1[e][:m * d * d * 4])     # final Gram matrices
            if kmode == kvc.KVC_FIT_FAST:
                assert torch.equal(kvc.kvc_fit_solver(caches[e + 1], sub), kvc.kvc_fit_solver(caches[e + 1], ws1[e]))
                assert int((kvc.kvc_fit_solver(caches[e + 1], sub) == 0).sum()) == m
    # edges of different rank: served one by one inside the call, same results
    if kmode == kvc.KVC_FIT_FAST:
        def fresh_r(rr):
            return kvc.State(torch.zeros(L, H, T, rr, device=DEV), torch.zeros(L, H, T, rr, device=DEV),
                             torch.zeros(L, H, rr, d, device=DEV), torch.zeros(L, H, rr, d, device=DEV))
        ranks = (8, 16, 40)
        mixed = [fresh_r(rr) for rr in ranks]
        ws = torch.zeros(kvc.kvc_chain_update_workspace_bytes(caches, mixed, kmode), dtype=torch.uint8, device=DEV)
        kvc.kvc_state_update_chain(caches, pl, rope, mixed, kmode, workspace=ws)
        for e, rr in enumerate(ranks):
            ref = fresh_r(rr)
            w1 = torch.zeros(kvc.kvc_workspace_bytes(caches[e + 1], ref, kmode), dtype=torch.uint8, device=DEV)
            kvc.kvc_state_update(caches[e], caches[e + 1], pl[e + 1] - pl[e], rope, ref, kmode, workspace=w1)
            assert torch.equal(ref.basis_k, mixed[e].basis_k) and torch.equal(ref.coeff_v, mixed[e].coeff_v), rr
    # too small a workspace, too many agents: refused before anything runs
    if kmode != kvc.KVC_PROJECT:
        with pytest.raises(kvc.KvcError):
            kvc.kvc_state_update_chain(caches, pl, rope, allst, kmode, workspace=wsn[:total - 256])
