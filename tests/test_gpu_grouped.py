"""GPU parity of the per-layer feature grouping (D = H d, Sec. 3.1): one state per layer whose
coefficients are shared by the KV heads.  The oracle expands the grouped state into the
per-(layer, head) form (the two define the same low-rank product) and applies / projects as usual."""
import numpy as np
import pytest
import torch

import paper_2609_34060_b200 as kvc
from paper_2609_34060_b200 import workloads as wl
from oracle import kvc_oracle as orc

import helpers as hp

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

CFG_S = wl.CONFIGS["llama8b_8k"].scaled(name="8b_small", L=2, H=4, T=900)
CFG_P = wl.CONFIGS["vlm_16k"].scaled(name="vlm_small", L=2, H=2, T=1301, image_spans=())
CFG_R64 = wl.CONFIGS["llama70b_32k"].scaled(name="r64_small", L=1, H=3, T=515)
CFG_T = wl.CONFIGS["tiny"]

PATHS = [kvc.KVC_PATH_GENERIC, kvc.KVC_PATH_AUTO]
PATH_IDS = ["generic", "auto"]


@pytest.fixture(autouse=True)
def _reset_path():
    kvc.kvc_status_reset()
    yield
    kvc.kvc_set_path(kvc.KVC_PATH_AUTO)
    assert kvc.kvc_status_poll() == 0


def _grouped_state(cfg, hop, n_cov=None, basis_dtype=torch.float32):
    """Seeded draws: coefficients [L, n_cov, r], orthonormal basis rows in R^{H d} as [L, r, H d]."""
    n = cfg.T if n_cov is None else n_cov
    one = cfg.scaled(H=1, d=cfg.H * cfg.d)              # the generator's per-"head" draw at D = H d
    ck = wl.coefficients(cfg.L, 1, cfg.T, cfg.r, cfg.seed, 4 * hop + 0, "cpu")[:, 0, :n].contiguous()
    cv = wl.coefficients(cfg.L, 1, cfg.T, cfg.r, cfg.seed, 4 * hop + 1, "cpu")[:, 0, :n].contiguous()
    bk = wl.orthonormal_basis(cfg.L, 1, cfg.r, one.d, cfg.seed, 4 * hop + 2, "cpu")[:, 0].contiguous().to(basis_dtype)
    bv = wl.orthonormal_basis(cfg.L, 1, cfg.r, one.d, cfg.seed, 4 * hop + 3, "cpu")[:, 0].contiguous().to(basis_dtype)
    return kvc.State(ck, cv, bk, bv, n_cov=n, grouping=kvc.KVC_GROUP_LAYER)


def _oracle_state(cfg, st):
    f = lambda t: t.to(torch.float32).numpy()
    return orc.ungroup_state(f(st.coeff_k), f(st.coeff_v), f(st.basis_k), f(st.basis_v), cfg.H, n_cov=st.n_cov)


def _check(dst, odst, ref_k, ref_v):
    gk, gv = hp.logical_bits(dst, "k"), hp.logical_bits(dst, "v")
    assert hp.tol_ratio(gk, ref_k) <= 1.0 and hp.tol_ratio(gv, ref_v) <= 1.0
    assert hp.ulp_mismatch_fraction(gk, hp.logical_bits(odst, "k")) < 1e-2
    assert hp.ulp_mismatch_fraction(gv, hp.logical_bits(odst, "v")) < 1e-2


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
@pytest.mark.parametrize("cfg", [CFG_S, CFG_P, CFG_R64, CFG_T], ids=lambda c: c.name)
def test_grouped_apply(cfg, path):
    kvc.kvc_set_path(path)
    src_cpu = hp.make_cache(cfg)
    for n_cov, shift in ((cfg.T, 77), (cfg.T // 2 + 3, 0)):
        st = _grouped_state(cfg, 1, n_cov=n_cov)
        src = hp.to_dev(src_cpu, DEV)
        dst = hp.empty_dst(src_cpu, cfg, DEV, fill=3.0)
        kvc.kvc_apply(src, hp.state_to_dev(st, DEV), shift, kvc.Rope(cfg.theta), dst)
        torch.cuda.synchronize()
        if path == kvc.KVC_PATH_AUTO and cfg.d == 128:
            assert kvc.kvc_last_path() == kvc.KVC_PATH_TC
        osrc = hp.oracle_cache(src_cpu)
        odst = osrc.empty_like(page_table=None if dst.page_table is None else dst.page_table.cpu().numpy())
        odst, rk, rv = orc.apply(osrc, _oracle_state(cfg, st), shift, hp.inv_freq(cfg), dst=odst, want_ref=True)
        _check(dst, odst, rk, rv)


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_grouped_chain_and_batch(path):
    cfg = CFG_S.scaled(T=400)
    kvc.kvc_set_path(path)
    rope = kvc.Rope(cfg.theta)
    pl = [100, 180, 140]
    src_cpu = hp.make_cache(cfg)
    src = hp.to_dev(src_cpu, DEV)
    states = [_grouped_state(cfg, a) for a in (1, 2)]
    dev_states = [hp.state_to_dev(s, DEV) for s in states]
    outs = [hp.empty_dst(src_cpu, cfg, DEV) for _ in range(2)]
    kvc.kvc_chain(src, pl, dev_states, rope, outs)
    torch.cuda.synchronize()
    ocur = hp.oracle_cache(src_cpu)
    for a in (1, 2):
        onext, rk, rv = orc.apply(ocur, _oracle_state(cfg, states[a - 1]), pl[a] - pl[a - 1], hp.inv_freq(cfg), want_ref=True)
        if a == 1:
            _check(outs[0], onext, rk, rv)
        ocur = onext
    # the chain equals its hops one by one, bit for bit; a ragged batch of the same hops too
    one = hp.empty_dst(src_cpu, cfg, DEV)
    kvc.kvc_apply(outs[0], dev_states[1], pl[2] - pl[1], rope, one)
    torch.cuda.synchronize()
    assert torch.equal(one.k, outs[1].k) and torch.equal(one.v, outs[1].v)
    bd = [hp.empty_dst(src_cpu, cfg, DEV) for _ in range(2)]
    items = [kvc.Item(src, bd[0], dev_states[0], pl[1] - pl[0]), kvc.Item(outs[0], bd[1], dev_states[1], pl[2] - pl[1])]
    nb = kvc.kvc_batch_workspace_bytes(2)
    ws = torch.empty(nb, dtype=torch.uint8, device=DEV)
    stg = torch.empty(nb, dtype=torch.uint8).pin_memory()
    kvc.kvc_apply_batch(items, rope, ws, stg)
    torch.cuda.synchronize()
    assert torch.equal(bd[0].k, outs[0].k) and torch.equal(bd[1].v, outs[1].v)
    # the first hop once more as two items with token ranges over the same caches (the grouped coefficient rows are
    # addressed by absolute token): the same bits as the whole-cache item
    cut = 256
    tw = hp.empty_dst(src_cpu, cfg, DEV)
    parts = [kvc.Item(src, tw, dev_states[0], pl[1] - pl[0], 0, cut), kvc.Item(src, tw, dev_states[0], pl[1] - pl[0], cut, cfg.T)]
    kvc.kvc_apply_batch(parts, rope, ws, stg)
    torch.cuda.synchronize()
    assert torch.equal(tw.k, outs[0].k) and torch.equal(tw.v, outs[0].v)


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
@pytest.mark.parametrize("cfg", [CFG_S, CFG_P, CFG_T], ids=lambda c: c.name)
def test_grouped_project(cfg, path):
    """coeff[l, t, :] = sum over heads of (tgt - Rot(src))[l, h, t, :] . basis[l][:, h d : (h+1) d]^T."""
    kvc.kvc_set_path(path)
    rope = kvc.Rope(cfg.theta)
    inv = hp.inv_freq(cfg)
    shift = 51
    src_cpu = hp.make_cache(cfg)
    tgt_cpu = hp.make_cache(cfg.scaled(seed=cfg.seed + 3))
    if src_cpu.page_table is not None:       # same geometry, another table
        tgt_cpu = hp.make_cache(cfg.scaled(seed=cfg.seed + 3), table_tag=9)
    given = _grouped_state(cfg, 2)
    n = cfg.T - 37
    st = kvc.State(torch.full((cfg.L, n, cfg.r), 7.0, device=DEV), torch.full((cfg.L, n, cfg.r), 7.0, device=DEV),
                   given.basis_k.to(DEV), given.basis_v.to(DEV), n_cov=n, grouping=kvc.KVC_GROUP_LAYER)
    kvc.kvc_state_update(hp.to_dev(src_cpu, DEV), hp.to_dev(tgt_cpu, DEV), shift, rope, st, kvc.KVC_PROJECT)
    torch.cuda.synchronize()
    if path == kvc.KVC_PATH_AUTO and cfg.d == 128:
        assert kvc.kvc_last_path() == kvc.KVC_PATH_TC
    osrc, otgt = hp.oracle_cache(src_cpu), hp.oracle_cache(tgt_cpu)
    for which, got, basis in (("k", st.coeff_k, given.basis_k), ("v", st.coeff_v, given.basis_v)):
        g = got.cpu().numpy().astype(np.float64)
        for l in range(cfg.L):
            deltas = [orc.deviation(osrc.get_bits(which, l, h), otgt.get_bits(which, l, h), shift, inv, which == "k")[:n]
                      for h in range(cfg.H)]
            ref = orc.project_grouped(deltas, basis[l].numpy())
            # the per-head bound of the projection, summed over the heads
            bn = np.linalg.norm(basis[l].numpy().astype(np.float64).reshape(cfg.r, cfg.H, cfg.d), axis=2)   # [r, H]
            tol = 1e-6 * np.ones_like(ref)
            for h in range(cfg.H):
                xs = np.linalg.norm(orc.bf16_to_f64(osrc.get_bits(which, l, h))[:n], axis=1)
                xt = np.linalg.norm(orc.bf16_to_f64(otgt.get_bits(which, l, h))[:n], axis=1)
                dn = np.linalg.norm(deltas[h], axis=1)
                tol += (2.0 ** -12 * dn + 2.0 ** -18 * (xs + xt))[:, None] * bn[None, :, h]
            assert np.all(np.abs(g[l] - ref) <= tol), (which, l, float(np.max(np.abs(g[l] - ref) / tol)))


def _grouped_edge(cfg, sigma, hop=1):
    """Source and target of one edge whose deviation has rank r on the concatenated feature axis
    (D = H d): target = bf16(Align(src) + c B + sigma noise) with B [r, H d] orthonormal rows, built by
    the oracle from generator draws.  Also the oracle's unrounded Align(src) + c B."""
    src_cpu = hp.make_cache(cfg)
    true = _grouped_state(cfg, hop)
    pl = wl.prefix_lengths(cfg)
    shift = pl[hop] - pl[hop - 1]
    nk = wl.noise((cfg.L, cfg.H, cfg.T, cfg.d), cfg.seed, 2 * hop).numpy()
    nv = wl.noise((cfg.L, cfg.H, cfg.T, cfg.d), cfg.seed, 2 * hop + 1).numpy()
    osrc = hp.oracle_cache(src_cpu)
    ost = _oracle_state(cfg, true)
    otgt = orc.make_target(osrc, ost, shift, hp.inv_freq(cfg), nk, nv, sigma)
    as_t = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
    if cfg.paged:
        tgt_cpu = kvc.Cache(as_t(otgt.k), as_t(otgt.v), T=cfg.T, page_table=src_cpu.page_table)
    else:
        tgt_cpu = kvc.Cache(as_t(otgt.k), as_t(otgt.v))
    return src_cpu, tgt_cpu, osrc, otgt, ost, shift


def _fit_grouped(src, tgt, shift, cfg, r, mode):
    L, H, T, d = cfg.L, cfg.H, cfg.T, cfg.d
    st = kvc.State(torch.zeros(L, T, r, device=DEV), torch.zeros(L, T, r, device=DEV),
                   torch.full((L, r, H * d), 3.0, device=DEV), torch.full((L, r, H * d), 3.0, device=DEV),
                   grouping=kvc.KVC_GROUP_LAYER)
    ws = torch.zeros(kvc.kvc_workspace_bytes(tgt, st, mode), dtype=torch.uint8, device=DEV)
    kvc.kvc_state_update(src, tgt, shift, kvc.Rope(cfg.theta), st, mode, workspace=ws)
    torch.cuda.synchronize()
    return st, ws


CFG_G2 = wl.CONFIGS["llama8b_8k"].scaled(name="8b_H2", L=2, H=2, T=700, r=16)
CFG_G8 = wl.CONFIGS["llama8b_8k"].scaled(name="8b_H8", L=1, H=8, T=1100)           # D = 1024, r = 32
CFG_GP = wl.CONFIGS["vlm_16k"].scaled(name="vlm_H4", L=1, H=4, T=901, image_spans=())  # paged, D = 512
CFG_G64 = wl.CONFIGS["tiny"].scaled(name="tiny_d64", L=2, H=3, T=333)                  # head_dim 64: D = 192, the CUDA-core
                                                                                        # passes; 48 columns per block of a cluster


@pytest.mark.parametrize("cfg", [CFG_G2, CFG_G8, CFG_GP, CFG_G64], ids=lambda c: c.name)
@pytest.mark.parametrize("mode", ["fit", "fit_fast"])
def test_grouped_fit(cfg, mode):
    """FIT under D = H d (Sec. 3.1, Eq. 7): the r leading right singular vectors of a layer's concatenated
    deviation.  Against the oracle's concatenated deviation: eigenvalues from a library routine on its
    Gram matrix, the leading subspace's projector, orthonormal rows with the sign rule, the Eckart-Young
    residual of coeff . basis, coefficient columns orthogonal with the eigenvalues as energies."""
    kmode = kvc.KVC_FIT if mode == "fit" else kvc.KVC_FIT_FAST
    src_cpu, tgt_cpu, osrc, otgt, ost, shift = _grouped_edge(cfg, cfg.sigma)
    src, tgt = hp.to_dev(src_cpu, DEV), hp.to_dev(tgt_cpu, DEV)
    r, D = cfg.r, cfg.H * cfg.d
    st, ws = _fit_grouped(src, tgt, shift, cfg, r, kmode)
    assert kvc.kvc_status_poll() == 0
    assert bool((kvc.kvc_group_fit_solver(tgt, ws) == kvc.KVC_SOLVER_SUBSPACE).all())
    ev = kvc.kvc_group_fit_eigenvalues(tgt, ws).cpu().numpy().astype(np.float64)
    f = hp.inv_freq(cfg)
    for l in range(cfg.L):
        for i, (which, B_t, c_t) in enumerate((("k", st.basis_k, st.coeff_k), ("v", st.basis_v, st.coeff_v))):
            cat = np.concatenate([orc.deviation(osrc.get_bits(which, l, h), otgt.get_bits(which, l, h), shift, f, which == "k")
                                  for h in range(cfg.H)], axis=1)                       # [T, H d]
            G = orc.gram(cat)
            w, V = np.linalg.eigh(G)
            w, V = w[::-1], V[:, ::-1]
            e = ev[l, i]
            assert np.max(np.abs(e[:r] - w[:r])) <= 2e-4 * w[0]
            assert np.allclose(e[r:], e[r]) and e[r] <= e[r - 1]
            assert abs(np.sum(e) - np.sum(w)) <= 2e-4 * np.sum(w)                       # the trace
            B = B_t[l].cpu().numpy().astype(np.float64)
            c = c_t[l].cpu().numpy().astype(np.float64)
            assert np.max(np.abs(B @ B.T - np.eye(r))) <= 2e-5
            assert np.all(B[np.arange(r), np.argmax(np.abs(B), axis=1)] > 0)
            assert np.linalg.norm(B.T @ B - V[:, :r] @ V[:, :r].T) <= 1e-2
            tail = float(np.sum(w[r:]))
            res = float(np.sum((cat - c @ B) ** 2))
            assert res <= 1.001 * tail + 1e-6 * float(np.sum(w)), (res, tail)
            Gc = c.T @ c
            assert np.max(np.abs(Gc - np.diag(np.diag(Gc)))) <= 2e-3 * w[0]
            assert np.max(np.abs(np.diag(Gc) - w[:r])) <= 1e-3 * w[0]
            # every row is an eigenvector of the oracle's Gram matrix to the solver's stated level
            assert np.max(np.linalg.norm(G @ B.T - B.T * np.diag(B @ G @ B.T)[None, :], axis=0)) <= 4e-4 * w[0]


@pytest.mark.parametrize("cfg", [CFG_G2, CFG_G8], ids=lambda c: c.name)
def test_grouped_update_then_apply_round_trip(cfg):
    """A rank-r deviation across the heads, fitted under grouping and applied again, gives back the
    target up to the noise floor and the bf16 roundings (the bound of the per-head round trip: the
    target's own rounding error, large in the outlier channels, is part of the fitted deviation and
    comes back through the coefficients)."""
    src_cpu, tgt_cpu, osrc, otgt, ost, shift = _grouped_edge(cfg, cfg.sigma)
    src, tgt = hp.to_dev(src_cpu, DEV), hp.to_dev(tgt_cpu, DEV)
    st, ws = _fit_grouped(src, tgt, shift, cfg, cfg.r, kvc.KVC_FIT)
    assert kvc.kvc_status_poll() == 0
    dst = hp.empty_dst(src_cpu, cfg, DEV)
    kvc.kvc_apply(src, st, shift, kvc.Rope(cfg.theta), dst)
    torch.cuda.synchronize()
    for which in ("k", "v"):
        got = orc.bf16_to_f64(hp.logical_bits(dst, which))
        want = orc.bf16_to_f64(hp.logical_bits(otgt, which))
        err = np.abs(got - want)
        assert np.mean(err > 2.0 ** -6 * np.abs(want) + 0.02) < 1e-3
        assert np.max(err) <= 2.0 ** -4 * np.max(np.abs(want))


def test_grouped_fit_without_a_gap_is_flagged_and_zero_is_zero():
    """A flat spectrum (a Gaussian cache factorised by itself) has no gap behind the r-th eigenvalue: the
    rows come back orthonormal, the matrix's code names the reason and KVC_FLAG_NOT_CONVERGED is raised
    (there is no second solver at D = H d).  An all-zero deviation gives a zero state without a flag."""
    cfg = CFG_G2.scaled(T=400, r=8)
    src = hp.to_dev(hp.make_cache(cfg), DEV)
    st, ws = _fit_grouped(None, src, 0, cfg, 8, kvc.KVC_FIT_FAST)
    codes = kvc.kvc_group_fit_solver(src, ws).cpu().numpy()
    assert np.all(codes[:, 1] > 0), codes                 # values: no structure at all
    assert kvc.kvc_status_poll() & kvc.KVC_FLAG_NOT_CONVERGED
    kvc.kvc_status_reset()
    B = st.basis_v[0].cpu().numpy().astype(np.float64)
    assert np.max(np.abs(B @ B.T - np.eye(8))) <= 1e-4
    z = kvc.Cache(torch.zeros_like(src.k), torch.zeros_like(src.v))
    st, ws = _fit_grouped(None, z, 0, cfg, 8, kvc.KVC_FIT)
    assert kvc.kvc_status_poll() == 0
    assert np.all(kvc.kvc_group_fit_solver(z, ws).cpu().numpy() == kvc.KVC_SOLVER_FULL_DEPENDENT)
    assert torch.all(st.basis_k == 0) and torch.all(st.coeff_v == 0)
    assert float(kvc.kvc_group_fit_eigenvalues(z, ws).abs().max()) == 0.0


def _expand(cfg, g):
    """The per-(layer, head) state that defines the same low-rank product as the grouped state g."""
    L, H, d, r = cfg.L, cfg.H, cfg.d, g.r
    ex = lambda c: c[:, None].expand(L, H, c.shape[1], r).contiguous()
    sp = lambda b: b.to(torch.float32).view(L, r, H, d).permute(0, 2, 1, 3).contiguous()
    return kvc.State(ex(g.coeff_k), ex(g.coeff_v), sp(g.basis_k), sp(g.basis_v), n_cov=g.n_cov)


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_grouped_anchors_in_gate_token_weights_and_multi_apply(path):
    """Anchor pools whose states are grouped by layer (one of the three per head, to show that pools may
    mix): gate distances (Eq. 9), token-wise weights (App. A.3) and the weighted multi-anchor apply (Eq. 8),
    each against the oracle run on the expanded per-head form of the same states."""
    from test_gpu_gate import _oracle_dist
    from test_gpu_multi import _oracle, _oracle_token_weights, _weights, _check as _check_multi
    cfg = CFG_S.scaled(T=777)
    L, H, T, d = cfg.L, cfg.H, cfg.T, cfg.d
    grouped = [_grouped_state(cfg, 1), _grouped_state(cfg, 2, n_cov=T - 130), hp.make_state(cfg, 3)]
    per_head = [_expand(cfg, grouped[0]), _expand(cfg, grouped[1]), grouped[2]]
    anchor_pos, src_pos = [100, 37, 412], 250
    # the source cache: close to anchor 0's reconstruction (keys moved to the source's positions), oracle arithmetic
    src_cpu = hp.make_cache(cfg)
    osrc = hp.oracle_cache(src_cpu)
    inv = hp.inv_freq(cfg)
    eps = wl.noise((2, L, H, T, d), cfg.seed, 91, "cpu").numpy().astype(np.float64)
    for l in range(L):
        for h in range(H):
            for wi, which in enumerate(("k", "v")):
                c = getattr(per_head[0], "coeff_" + which)[l, h].numpy().astype(np.float64)
                b = getattr(per_head[0], "basis_" + which)[l, h].numpy().astype(np.float64)
                x = c @ b
                if which == "k":
                    x = orc.rope_shift(x, src_pos - anchor_pos[0], inv)
                osrc.put_bits(which, l, h, orc.f64_to_bf16_bits(x + 0.2 * eps[wi, l, h]))
    mk = lambda a: torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16)
    src_cpu = kvc.Cache(mk(osrc.k), mk(osrc.v))
    src = hp.to_dev(src_cpu, DEV)
    dev = [hp.state_to_dev(a, DEV) for a in grouped]
    kvc.kvc_set_path(path)
    # ---- gate distance at a length every anchor covers
    k = T - 200
    d2 = torch.full((3,), -1.0, dtype=torch.float64, device=DEV)
    kvc.kvc_gate_distance(src, dev, k, d2)
    torch.cuda.synchronize()
    ref = _oracle_dist(cfg, osrc, per_head, k)
    assert np.all(np.abs(np.sqrt(d2.cpu().numpy()) - ref) <= 1e-4 * ref + 1e-6), (d2, ref)
    if path != kvc.KVC_PATH_AUTO:
        return                                   # token weights and the multi-anchor apply are tensor-core kernels
    # ---- token weights
    tp = kvc.kvc_multi_tpad(T)
    wk, wv = torch.full((3, tp), -1.0, device=DEV), torch.full((3, tp), -1.0, device=DEV)
    ws = torch.empty(kvc.kvc_token_weights_workspace_bytes(src, 3), dtype=torch.uint8, device=DEV)
    kvc.kvc_token_weights(src, src_pos, dev, anchor_pos, kvc.Rope(cfg.theta), wk, wv, ws)
    torch.cuda.synchronize()
    rk, rv = _oracle_token_weights(cfg, osrc, src_pos, per_head, anchor_pos)
    gk, gv = wk.cpu().numpy().astype(np.float64), wv.cpu().numpy().astype(np.float64)
    assert np.max(np.abs(gk[:, :T] - rk)) <= 2e-5 and np.max(np.abs(gv[:, :T] - rv)) <= 2e-5
    # ---- weighted multi-anchor apply with seeded weights
    w_k, w_v = _weights(3, T, cfg.seed, 1), _weights(3, T, cfg.seed, 2)
    shift = -41
    dst = hp.empty_dst(src_cpu, cfg, DEV, fill=-7.0)
    ws2 = torch.empty(max(kvc.kvc_multi_workspace_bytes(src, dev), 128), dtype=torch.uint8, device=DEV)
    kvc.kvc_apply_multi(src, dev, w_k.to(DEV), w_v.to(DEV), shift, kvc.Rope(cfg.theta), dst, ws2)
    torch.cuda.synchronize()
    odst, ref_k, ref_v = _oracle(cfg, src_cpu, per_head, w_k, w_v, shift)
    _check_multi(dst, odst, ref_k, ref_v)


def test_grouped_fit_beyond_rank_32_is_rejected():
    cfg = CFG_S.scaled(T=200)
    src = hp.to_dev(hp.make_cache(cfg), DEV)
    ws = torch.empty(1 << 26, dtype=torch.uint8, device=DEV)
    big = _grouped_state(cfg.scaled(r=64), 1)            # the grouped fit serves r <= 32
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_state_update(None, src, 0, kvc.Rope(cfg.theta), hp.state_to_dev(big, DEV), kvc.KVC_FIT, workspace=ws)
    assert e.value.code == kvc.KVC_E_UNSUPPORTED
