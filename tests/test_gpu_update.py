"""GPU parity of kvc_state_update (project and fit modes) against the fp64 oracle.

Coefficients with a *given* basis are compared element by element.  A fitted basis is not
unique (sign, rotations inside near-equal singular values), so fit mode is checked through
what is unique: the Gram matrix, the eigenvalues, orthonormality, the projector on a
well-separated spectrum, the Eckart-Young residual and the update -> apply round trip.
"""
import numpy as np
import pytest
import torch

import paper_2609_34060_b200 as kvc
from paper_2609_34060_b200 import workloads as wl
from oracle import kvc_oracle as orc

import helpers as hp

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

CFG_TINY = wl.CONFIGS["tiny"]
CFG_8B_S = wl.CONFIGS["llama8b_8k"].scaled(name="8b_small", L=2, H=2, T=700)
CFG_VLM_S = wl.CONFIGS["vlm_16k"].scaled(name="vlm_small", L=1, H=2, T=1003, image_spans=((512, 1024),))
CFG_R64_S = wl.CONFIGS["llama70b_32k"].scaled(name="r64_small", L=1, H=2, T=390)

PATHS = [kvc.KVC_PATH_GENERIC, kvc.KVC_PATH_AUTO]
PATH_IDS = ["generic", "auto"]


@pytest.fixture(autouse=True)
def _reset_path():
    kvc.kvc_status_reset()
    yield
    kvc.kvc_set_path(kvc.KVC_PATH_AUTO)
    assert kvc.kvc_status_poll() == 0


def _edge(cfg, hop=1):
    """(src, tgt) caches of one edge on the CPU, the true state, the shift.  The target is
    derived by the oracle from generator draws: bf16(Align(src) + A B + sigma noise)."""
    src_cpu = hp.make_cache(cfg)
    true = hp.make_state(cfg, hop)
    pl = wl.prefix_lengths(cfg)
    shift = pl[hop] - pl[hop - 1]
    nk = wl.noise((cfg.L, cfg.H, cfg.T, cfg.d), cfg.seed, 2 * hop).numpy()
    nv = wl.noise((cfg.L, cfg.H, cfg.T, cfg.d), cfg.seed, 2 * hop + 1).numpy()
    osrc = hp.oracle_cache(src_cpu)
    otgt = orc.make_target(osrc, hp.oracle_state(true), shift, hp.inv_freq(cfg), nk, nv, cfg.sigma)
    as_t = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
    if cfg.paged:
        tgt_cpu = kvc.Cache(as_t(otgt.k), as_t(otgt.v), T=cfg.T, page_table=src_cpu.page_table)
    else:
        tgt_cpu = kvc.Cache(as_t(otgt.k), as_t(otgt.v))
    return src_cpu, tgt_cpu, osrc, otgt, true, shift


def _coeff_tol(osrc, otgt, delta, basis, l, h, which):
    """|c_gpu - c_ref| <= 2^-12 |Delta_t| |B_q| + 2^-18 (|src_t| + |tgt_t|) |B_q| + 1e-6.
    First term: product rounding of the split-precision contraction; second: float32
    rotation and cancellation in tgt - Rot(src), relative to the inputs' size."""
    n = delta.shape[0]
    bn = np.linalg.norm(basis, axis=1)[None, :]
    dn = np.linalg.norm(delta, axis=1)[:, None]
    sn = np.linalg.norm(orc.bf16_to_f64(osrc.get_bits(which, l, h)), axis=1)[:n, None] if osrc is not None else 0.0
    tn = np.linalg.norm(orc.bf16_to_f64(otgt.get_bits(which, l, h)), axis=1)[:n, None]
    return 2.0 ** -12 * dn * bn + 2.0 ** -18 * (sn + tn) * bn + 1e-6


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
@pytest.mark.parametrize("cfg", [CFG_TINY, CFG_8B_S, CFG_VLM_S, CFG_R64_S], ids=lambda c: c.name)
def test_project_mode(cfg, path):
    src_cpu, tgt_cpu, osrc, otgt, true, shift = _edge(cfg)
    n_cov = cfg.T - 5
    # project onto a basis that is NOT the true one (any given basis must work)
    other = hp.make_state(cfg, 3)
    ost, _ = orc.state_update(osrc, otgt, shift, hp.inv_freq(cfg), mode=orc.PROJECT, n_cov=n_cov,
                              basis_k=other.basis_k.numpy(), basis_v=other.basis_v.numpy())
    kvc.kvc_set_path(path)
    src, tgt = hp.to_dev(src_cpu, DEV), hp.to_dev(tgt_cpu, DEV)
    st = kvc.State(torch.full((cfg.L, cfg.H, n_cov, cfg.r), 7.0, device=DEV),
                   torch.full((cfg.L, cfg.H, n_cov, cfg.r), 7.0, device=DEV),
                   other.basis_k.to(DEV), other.basis_v.to(DEV), n_cov=n_cov)
    kvc.kvc_state_update(src, tgt, shift, kvc.Rope(cfg.theta), st, kvc.KVC_PROJECT)
    torch.cuda.synchronize()
    if path == kvc.KVC_PATH_AUTO and cfg.d == 128:
        assert kvc.kvc_last_path() == kvc.KVC_PATH_TC, "the TMA + tcgen05 kernels should have served this call"
    ck, cv = st.coeff_k.cpu().numpy().astype(np.float64), st.coeff_v.cpu().numpy().astype(np.float64)
    worst = 0.0
    for l in range(cfg.L):
        for h in range(cfg.H):
            for which, got, ref, bs in (("k", ck, ost.coeff_k, other.basis_k), ("v", cv, ost.coeff_v, other.basis_v)):
                dl = orc.deviation(osrc.get_bits(which, l, h), otgt.get_bits(which, l, h), shift, hp.inv_freq(cfg),
                                   which == "k")[:n_cov]
                tol = _coeff_tol(osrc, otgt, dl, bs[l, h].numpy().astype(np.float64), l, h, which)
                worst = max(worst, float(np.max(np.abs(got[l, h] - ref[l, h].astype(np.float64)) / tol)))
    assert worst <= 1.0, worst
    # inputs are only read
    assert torch.equal(src.k.cpu(), src_cpu.k) and torch.equal(tgt.v.cpu(), tgt_cpu.v)


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_project_without_source_and_bf16_basis(path):
    cfg = CFG_8B_S.scaled(T=200)
    src_cpu, tgt_cpu, osrc, otgt, true, shift = _edge(cfg)
    other = hp.make_state(cfg, 3, basis_dtype=torch.bfloat16)
    ost, _ = orc.state_update(None, otgt, 0, hp.inv_freq(cfg), mode=orc.PROJECT,
                              basis_k=other.basis_k.float().numpy(), basis_v=other.basis_v.float().numpy())
    kvc.kvc_set_path(path)
    st = kvc.State(torch.zeros(cfg.L, cfg.H, cfg.T, cfg.r, device=DEV), torch.zeros(cfg.L, cfg.H, cfg.T, cfg.r, device=DEV),
                   other.basis_k.to(DEV), other.basis_v.to(DEV))
    kvc.kvc_state_update(None, hp.to_dev(tgt_cpu, DEV), 0, kvc.Rope(cfg.theta), st, kvc.KVC_PROJECT)
    torch.cuda.synchronize()
    for got, ref in ((st.coeff_k, ost.coeff_k), (st.coeff_v, ost.coeff_v)):
        err = np.abs(got.cpu().numpy().astype(np.float64) - ref.astype(np.float64))
        # Delta = tgt: |c| up to ~|tgt_t|; float32 accumulation over d terms
        assert np.max(err) <= 2.0 ** -12 * 40.0


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
@pytest.mark.parametrize("cfg", [CFG_TINY, CFG_8B_S.scaled(T=520), CFG_VLM_S.scaled(T=400, image_spans=())],
                         ids=lambda c: c.name)
def test_fit_mode(cfg, path):
    src_cpu, tgt_cpu, osrc, otgt, true, shift = _edge(cfg)
    f = hp.inv_freq(cfg)
    ost, oev = orc.state_update(osrc, otgt, shift, f, r=cfg.r, mode=orc.FIT)
    kvc.kvc_set_path(path)
    src, tgt = hp.to_dev(src_cpu, DEV), hp.to_dev(tgt_cpu, DEV)
    L, H, T, d, r = cfg.L, cfg.H, cfg.T, cfg.d, cfg.r
    st = kvc.State(torch.zeros(L, H, T, r, device=DEV), torch.zeros(L, H, T, r, device=DEV),
                   torch.zeros(L, H, r, d, device=DEV), torch.zeros(L, H, r, d, device=DEV))
    ws = torch.empty(kvc.kvc_workspace_bytes(tgt, st, kvc.KVC_FIT), dtype=torch.uint8, device=DEV)
    kvc.kvc_state_update(src, tgt, shift, kvc.Rope(cfg.theta), st, kvc.KVC_FIT, workspace=ws)
    torch.cuda.synchronize()
    wsf = ws.view(torch.float32).cpu().numpy().astype(np.float64)
    G = wsf[: L * H * 2 * d * d].reshape(L, H, 2, d, d)
    ev = wsf[2 * L * H * 2 * d * d: 2 * L * H * 2 * d * d + L * H * 2 * d].reshape(L, H, 2, d)
    for l in range(L):
        for h in range(H):
            for i, (which, B_t, c_t, B_o) in enumerate((("k", st.basis_k, st.coeff_k, ost.basis_k),
                                                        ("v", st.basis_v, st.coeff_v, ost.basis_v))):
                dl = orc.deviation(osrc.get_bits(which, l, h), otgt.get_bits(which, l, h), shift, f, which == "k")
                Gref = orc.gram(dl)
                dg = np.sqrt(np.diag(Gref))
                # float32 accumulation over T rows of split-precision products
                assert np.max(np.abs(G[l, h, i] - Gref) / (2.0 ** -12 * np.outer(dg, dg) + 1e-6)) <= 1.0
                w = oev[l, h, i]
                assert np.max(np.abs(ev[l, h, i] - w)) <= 1e-4 * w[0]
                assert np.all(np.diff(ev[l, h, i]) <= 1e-6 * w[0])                       # descending
                B = B_t[l, h].cpu().numpy().astype(np.float64)
                c = c_t[l, h].cpu().numpy().astype(np.float64)
                assert np.max(np.abs(B @ B.T - np.eye(r))) <= 1e-4                        # orthonormal rows
                assert np.all(B[np.arange(r), np.argmax(np.abs(B), axis=1)] > 0)          # sign convention
                # the spectrum is well separated at r (rank-r signal over a noise floor):
                # the projector is unique and must match the oracle's
                Bo = B_o[l, h].astype(np.float64)
                assert np.linalg.norm(B.T @ B - Bo.T @ Bo) <= 1e-2
                # Eckart-Young: no rank-r state reconstructs Delta better than the tail energy
                tail = float(np.sum(w[r:]))
                res = float(np.sum((dl - c @ B) ** 2))
                assert res <= 1.001 * tail + 1e-6 * float(np.sum(w)), (res, tail)
                # coeff columns are U_r Sigma_r: mutually orthogonal, energies = top eigenvalues
                Gc = c.T @ c
                assert np.max(np.abs(Gc - np.diag(np.diag(Gc)))) <= 2e-3 * w[0]
                assert np.max(np.abs(np.sort(np.diag(Gc))[::-1] - w[:r])) <= 1e-3 * w[0]
    # round trip: applying the fitted state to the source gives back the target (up to the
    # noise floor and bf16 rounding)
    dst = kvc.Cache(torch.zeros_like(src.k), torch.zeros_like(src.v), T=cfg.T if cfg.paged else None,
                    page_table=src.page_table)
    kvc.kvc_apply(src, st, shift, kvc.Rope(cfg.theta), dst)
    torch.cuda.synchronize()
    for which in ("k", "v"):
        got = orc.bf16_to_f64(hp.logical_bits(dst, which))
        want = orc.bf16_to_f64(hp.logical_bits(otgt, which))
        err = np.abs(got - want)
        assert np.mean(err > 2.0 ** -6 * np.abs(want) + 0.02) < 1e-3


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_fit_rank_limits(path):
    # fewer covered rows than the requested rank: the surplus basis rows are zero
    cfg = CFG_TINY.scaled(T=40, r=8)
    src_cpu, tgt_cpu, osrc, otgt, true, shift = _edge(cfg)
    kvc.kvc_set_path(path)
    src, tgt = hp.to_dev(src_cpu, DEV), hp.to_dev(tgt_cpu, DEV)
    n_cov = 5
    st = kvc.State(torch.zeros(cfg.L, cfg.H, n_cov, 8, device=DEV), torch.zeros(cfg.L, cfg.H, n_cov, 8, device=DEV),
                   torch.ones(cfg.L, cfg.H, 8, cfg.d, device=DEV), torch.ones(cfg.L, cfg.H, 8, cfg.d, device=DEV), n_cov=n_cov)
    ws = torch.empty(kvc.kvc_workspace_bytes(tgt, st, kvc.KVC_FIT), dtype=torch.uint8, device=DEV)
    kvc.kvc_state_update(src, tgt, shift, kvc.Rope(cfg.theta), st, kvc.KVC_FIT, workspace=ws)
    torch.cuda.synchronize()
    B = st.basis_k.cpu().numpy().astype(np.float64)
    assert np.all(B[:, :, n_cov:] == 0)
    assert np.max(np.abs(B[0, 0, :n_cov] @ B[0, 0, :n_cov].T - np.eye(n_cov))) <= 1e-4
    # with all five directions kept the five covered rows are reproduced exactly
    dl = orc.deviation(osrc.get_bits("k", 0, 0), otgt.get_bits("k", 0, 0), shift, hp.inv_freq(cfg), True)[:n_cov]
    c = st.coeff_k[0, 0].cpu().numpy().astype(np.float64)
    assert np.max(np.abs(c @ B[0, 0] - dl)) <= 1e-3 * np.max(np.abs(dl))


@pytest.mark.parametrize("base", [CFG_TINY.scaled(L=1, H=1, T=300), CFG_8B_S.scaled(L=1, H=1, T=300, r=8)],
                         ids=["d64", "d128"])
def test_fit_rank_sweep(base):
    """Fit ranks from 1 to 64 on a rank-8 deviation over a noise floor: ranks below, at and above the
    signal rank, on both sides of 32 (where the eigensolver changes its vector path).  Whatever the
    rank: orthonormal rows, the oracle's eigenvalues, no dependent-vector flag, and a residual at the
    tail energy (Eckart-Young).  A float32 reduction to tridiagonal form moves every eigenvalue by up
    to about d eps |T| (8e-6 |T| at d = 128), which is the size of the smallest eigenvalues kept at the
    larger ranks: each kept vector may miss that much energy, hence the allowance per vector."""
    src_cpu, tgt_cpu, osrc, otgt, true, shift = _edge(base)
    f = hp.inv_freq(base)
    src, tgt = hp.to_dev(src_cpu, DEV), hp.to_dev(tgt_cpu, DEV)
    T, d = base.T, base.d
    _, oev = orc.state_update(osrc, otgt, shift, f, r=8, mode=orc.FIT)
    for r in (1, 2, 3, 7, 8, 9, 31, 32, 33, 48, 64):
        st = kvc.State(torch.zeros(1, 1, T, r, device=DEV), torch.zeros(1, 1, T, r, device=DEV),
                       torch.zeros(1, 1, r, d, device=DEV), torch.zeros(1, 1, r, d, device=DEV))
        ws = torch.empty(kvc.kvc_workspace_bytes(tgt, st, kvc.KVC_FIT), dtype=torch.uint8, device=DEV)
        kvc.kvc_state_update(src, tgt, shift, kvc.Rope(base.theta), st, kvc.KVC_FIT, workspace=ws)
        torch.cuda.synchronize()
        ev = ws.view(torch.float32)[2 * 2 * d * d: 2 * 2 * d * d + 2 * d].cpu().numpy().astype(np.float64).reshape(2, d)
        for i, (which, B_t, c_t) in enumerate((("k", st.basis_k, st.coeff_k), ("v", st.basis_v, st.coeff_v))):
            dl = orc.deviation(osrc.get_bits(which, 0, 0), otgt.get_bits(which, 0, 0), shift, f, which == "k")
            w = oev[0, 0, i]
            assert np.max(np.abs(ev[i] - w)) <= 1e-4 * w[0], r
            B = B_t[0, 0].cpu().numpy().astype(np.float64)
            c = c_t[0, 0].cpu().numpy().astype(np.float64)
            assert np.max(np.abs(B @ B.T - np.eye(r))) <= 1e-4, r
            res = float(np.sum((dl - c @ B) ** 2))
            tail = float(np.sum(w[r:]))
            assert res <= tail + 8 * r * 1.2e-6 * w[0] + 1e-9 * float(np.sum(w)), (r, res, tail)
    assert kvc.kvc_status_poll() == 0


@pytest.mark.parametrize("d", [64, 128])
def test_fit_degenerate_spectra(d):
    """Spectra with a closed form, factorising a hand-made cache by itself (src = NULL).
    (a) All zeros: every eigenvalue 0, the basis rows and coefficients all zero, nothing flagged.
    (b) Token t carries the value 1 in dimension t mod 8 only: the Gram matrix is diag(T/8 x 8, 0, ...),
    an eight-fold eigenvalue.  At r = 8 the basis spans e_0..e_7 and reproduces the cache exactly; at
    r = 4 any orthonormal four-dimensional part of that span is right and leaves exactly half the energy;
    at r = 12 the four directions beyond the rank have eigenvalue zero: their rows are zero.
    (c) Two equal pairs and a single: singular values (3, 3, 2, 2, 1) on orthogonal +-1 patterns."""
    T = 256
    rope = kvc.Rope(10000.0)

    def fit(v_rows, r):
        cache = kvc.Cache(v_rows.to(torch.bfloat16).reshape(1, 1, T, d).contiguous().to(DEV),
                          v_rows.to(torch.bfloat16).reshape(1, 1, T, d).contiguous().to(DEV))
        st = kvc.State(torch.ones(1, 1, T, r, device=DEV), torch.ones(1, 1, T, r, device=DEV),
                       torch.ones(1, 1, r, d, device=DEV), torch.ones(1, 1, r, d, device=DEV))
        ws = torch.empty(kvc.kvc_workspace_bytes(cache, st, kvc.KVC_FIT), dtype=torch.uint8, device=DEV)
        kvc.kvc_state_update(None, cache, 0, rope, st, kvc.KVC_FIT, workspace=ws)
        torch.cuda.synchronize()
        ev = ws.view(torch.float32)[2 * 2 * d * d: 2 * 2 * d * d + 2 * d].cpu().numpy().astype(np.float64).reshape(2, d)
        return st, ev

    # (a)
    st, ev = fit(torch.zeros(T, d), 8)
    assert np.all(ev == 0)
    for t in (st.basis_k, st.basis_v, st.coeff_k, st.coeff_v):
        assert torch.all(t == 0)
    # (b)
    x = torch.zeros(T, d)
    x[torch.arange(T), torch.arange(T) % 8] = 1.0
    xn = x.numpy().astype(np.float64)
    for r in (4, 8, 12):
        st, ev = fit(x, r)
        for i, (B_t, c_t) in enumerate(((st.basis_k, st.coeff_k), (st.basis_v, st.coeff_v))):
            assert np.max(np.abs(ev[i, :8] - T / 8)) <= 1e-4 * T / 8 and np.max(np.abs(ev[i, 8:])) <= 1e-5 * T / 8
            B = B_t[0, 0].cpu().numpy().astype(np.float64)
            c = c_t[0, 0].cpu().numpy().astype(np.float64)
            k = min(r, 8)
            assert np.max(np.abs(B[:k] @ B[:k].T - np.eye(k))) <= 1e-5
            assert np.max(np.abs(B[:k, 8:])) <= 1e-5                     # inside span(e_0..e_7)
            assert np.all(B[k:] == 0) and np.all(c[:, k:] == 0)            # nothing beyond the rank of the data
            res = float(np.sum((xn - c @ B) ** 2))
            assert abs(res - (8 - k) * T / 8) <= 1e-4 * T, (r, res)
    # (c)
    had = np.array([[1 if bin(i & j).count("1") % 2 == 0 else -1 for j in range(8)] for i in range(8)], dtype=np.float64)
    u = np.repeat(had[:, :5], T // 8, axis=0) / np.sqrt(T)                 # orthonormal columns, entries +-1/16
    vt = np.zeros((5, d))
    for q in range(5):
        vt[q, 8 * q: 8 * q + 4] = 0.5                                      # orthonormal rows
    sv = np.array([3.0, 3.0, 2.0, 2.0, 1.0])
    y = (u * (16.0 * sv)) @ vt                                             # entries are small dyadic numbers: exact in bf16
    st, ev = fit(torch.from_numpy(y).float(), 5)
    want = np.concatenate([(16.0 * sv) ** 2, np.zeros(d - 5)])
    for i, (B_t, c_t) in enumerate(((st.basis_k, st.coeff_k), (st.basis_v, st.coeff_v))):
        assert np.max(np.abs(ev[i] - want)) <= 1e-4 * want[0]
        B = B_t[0, 0].cpu().numpy().astype(np.float64)
        c = c_t[0, 0].cpu().numpy().astype(np.float64)
        assert np.max(np.abs(B @ B.T - np.eye(5))) <= 1e-5
        assert np.max(np.abs(y - c @ B)) <= 1e-3
        # the single value's direction is unique up to sign; the pairs are planes
        assert abs(abs(B[4] @ vt[4]) - 1.0) <= 1e-4
        for pair in ((0, 1), (2, 3)):
            P = B[list(pair)]
            assert np.max(np.abs(P @ vt[list(pair)].T @ vt[list(pair)] - P)) <= 1e-3
    assert kvc.kvc_status_poll() == 0


@pytest.mark.parametrize("d", [64, 128])
def test_fit_clustered_spectra(d):
    """Twenty drawn spectra per head dimension with clusters of (nearly) equal singular values over a low
    floor, each factorised at one rank up to 32 and one above (the two vector paths of the eigensolver).
    Checked against a library eigensolver on the same bf16 data: eigenvalues, orthonormal rows at
    rounding level, a residual at the tail energy (allowance as in the rank sweep), nothing flagged, and
    as many live rows as there are eigenvalues the float32 solver can tell from zero."""
    T = 512
    for trial in range(20):
        x, _ = wl.clustered_rows(T, d, seed=11, tag=100 * d + trial)
        xn = x.to(torch.float64).numpy()
        w = np.linalg.eigvalsh(xn.T @ xn)[::-1]
        g = torch.Generator().manual_seed(1000 * d + trial)
        for r in (int(torch.randint(1, 33, (1,), generator=g)), int(torch.randint(33, min(d, 64) + 1, (1,), generator=g))):
            cache = kvc.Cache(x.reshape(1, 1, T, d).contiguous().to(DEV), x.reshape(1, 1, T, d).contiguous().to(DEV))
            st = kvc.State(torch.zeros(1, 1, T, r, device=DEV), torch.zeros(1, 1, T, r, device=DEV),
                           torch.zeros(1, 1, r, d, device=DEV), torch.zeros(1, 1, r, d, device=DEV))
            ws = torch.empty(kvc.kvc_workspace_bytes(cache, st, kvc.KVC_FIT), dtype=torch.uint8, device=DEV)
            kvc.kvc_state_update(None, cache, 0, kvc.Rope(10000.0), st, kvc.KVC_FIT, workspace=ws)
            torch.cuda.synchronize()
            assert kvc.kvc_status_poll() == 0, (trial, r)
            ev = ws.view(torch.float32)[2 * 2 * d * d + d: 2 * 2 * d * d + 2 * d].cpu().numpy().astype(np.float64)
            assert np.max(np.abs(ev - w)) <= 1e-4 * w[0], (trial, r)
            B = st.basis_v[0, 0].cpu().numpy().astype(np.float64)
            c = st.coeff_v[0, 0].cpu().numpy().astype(np.float64)
            live = np.abs(B).sum(axis=1) > 0
            k = int(live.sum())
            assert np.all(live[:k]) and k >= min(r, int(np.sum(w > 1e-5 * w[0]))), (trial, r, k)
            assert np.max(np.abs(B[:k] @ B[:k].T - np.eye(k))) <= 1e-5, (trial, r)
            res = float(np.sum((xn - c @ B) ** 2))
            assert res <= float(np.sum(w[k:])) + 8 * r * 1.2e-6 * w[0] + 1e-9 * float(np.sum(w)), (trial, r)


def test_effective_rank_from_fit_eigenvalues():
    """Sec. 3.1's diagnostic on the eigenvalues a FIT leaves behind: a deviation of exact rank 8 plus
    bf16 rounding noise has effective rank <= 8 at 90 % energy and matches the oracle's count on the
    oracle's eigenvalues; a flat Gaussian cache (base factorisation) needs most of its 128 directions."""
    cfg = wl.CONFIGS["llama8b_8k"].scaled(name="er", L=1, H=2, T=512, r=8)
    rope = kvc.Rope(cfg.theta)
    src_cpu = hp.make_cache(cfg)
    osrc = hp.oracle_cache(src_cpu)
    true = hp.make_state(cfg, hop=1)
    otgt = orc.apply(osrc, hp.oracle_state(true), 40, hp.inv_freq(cfg))
    mk = lambda a: torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16)
    src = hp.to_dev(src_cpu, DEV)
    tgt = kvc.Cache(mk(otgt.k).to(DEV), mk(otgt.v).to(DEV))
    L, H, T, d, r = cfg.L, cfg.H, cfg.T, cfg.d, cfg.r
    st = kvc.State(torch.empty(L, H, T, r, device=DEV), torch.empty(L, H, T, r, device=DEV),
                   torch.empty(L, H, r, d, device=DEV), torch.empty(L, H, r, d, device=DEV))
    ws = torch.empty(kvc.kvc_workspace_bytes(tgt, st, kvc.KVC_FIT), dtype=torch.uint8, device=DEV)
    kvc.kvc_state_update(src, tgt, 40, rope, st, kvc.KVC_FIT, workspace=ws)
    er = kvc.kvc_effective_rank(tgt, ws).cpu().numpy()
    _, ev = orc.state_update(osrc, otgt, 40, hp.inv_freq(cfg), r=r, mode=orc.FIT)
    for l in range(L):
        for h in range(H):
            for kv in range(2):
                want = orc.effective_rank(ev[l, h, kv])
                assert er[l, h, kv] == want and 1 <= want <= 8
    # base factorisation of the Gaussian cache itself: no low-rank structure
    kvc.kvc_state_update(None, src, 0, rope, st, kvc.KVC_FIT, workspace=ws)
    er = kvc.kvc_effective_rank(src, ws).cpu().numpy()
    for l in range(L):
        for h in range(H):
            v = orc.bf16_to_f64(osrc.get_bits("v", l, h))
            want = orc.effective_rank(np.linalg.eigvalsh(v.T @ v))
            assert abs(int(er[l, h, 1]) - want) <= 1 and want > 64      # a tie at the 90 % mark may fall either way
    assert kvc.kvc_effective_rank(src, ws, energy=1.0).max().item() <= d


def test_token_major_pages_update_gives_the_same_bits():
    """Pools whose pages are [page, H, d] instead of [H, page, d], described through the strides: projection and
    FIT_FAST give the same coefficients, bases and eigenvalues bit for bit."""
    cfg = CFG_VLM_S
    src_cpu, tgt_cpu, osrc, otgt, true, shift = _edge(cfg)
    src, tgt = hp.to_dev(src_cpu, DEV), hp.to_dev(tgt_cpu, DEV)
    tm = lambda t: t.permute(0, 1, 3, 2, 4).contiguous()
    as_tm = lambda c: kvc.Cache(tm(c.k), tm(c.v), T=cfg.T, page_table=c.page_table, token_major=True)
    src_t, tgt_t = as_tm(src), as_tm(tgt)
    L, H, T, d, r = cfg.L, cfg.H, cfg.T, cfg.d, cfg.r
    given = hp.make_state(cfg, 3)
    rope = kvc.Rope(cfg.theta)
    for mode in (kvc.KVC_PROJECT, kvc.KVC_FIT_FAST):
        outs = []
        for s_, t_ in ((src, tgt), (src_t, tgt_t)):
            st = kvc.State(torch.zeros(L, H, T, r, device=DEV), torch.zeros(L, H, T, r, device=DEV),
                           given.basis_k.to(DEV).clone(), given.basis_v.to(DEV).clone())
            ws = torch.zeros(max(kvc.kvc_workspace_bytes(t_, st, mode), 256), dtype=torch.uint8, device=DEV)
            kvc.kvc_state_update(s_, t_, shift, rope, st, mode, workspace=ws)
            torch.cuda.synchronize()
            assert kvc.kvc_last_path() == kvc.KVC_PATH_TC
            outs.append(st)
        a, b = outs
        assert torch.equal(a.coeff_k, b.coeff_k) and torch.equal(a.coeff_v, b.coeff_v)
        assert torch.equal(a.basis_k, b.basis_k) and torch.equal(a.basis_v, b.basis_v)
