"""Seeded sweep over random shapes: kvc_apply and kvc_state_update (project) against the fp64 oracle.

The other GPU tests pick their shapes by hand around known tile and page boundaries; this one
draws them (head_dim, rank, layers, heads, length, coverage, page size, shift, RoPE pairing,
basis dtype), so that combinations nobody thought of are compared element by element too.
Whatever kernel family the library chooses for a shape is the one that is checked.
The environment variable KVC_SWEEP_OFFSET (an integer, default 0) moves every draw to another part of
the seed space: the committed sweep is one sample, a campaign runs it at several offsets.
"""
import os

import numpy as np
import pytest
import torch

import paper_2609_34060_b200 as kvc
from paper_2609_34060_b200 import workloads as wl
from oracle import kvc_oracle as orc

import helpers as hp

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
BASE = wl.CONFIGS["llama8b_8k"]
SWEEP_OFFSET = int(os.environ.get("KVC_SWEEP_OFFSET", "0"))


@pytest.fixture(autouse=True)
def _clean_status():
    kvc.kvc_status_reset()
    kvc.kvc_set_path(kvc.KVC_PATH_AUTO)
    yield
    assert kvc.kvc_status_poll() == 0


def _draw(seed):
    g = np.random.default_rng(77000 + seed + 100000 * SWEEP_OFFSET)
    d = int(g.choice([64, 128, 128, 128]))
    r = int(g.choice([1, 3, 4, 8, 12, 16, 17, 24, 32, 33, 40, 48, 64]))
    T = int(g.choice([g.integers(1, 140), g.integers(140, 900)]))
    paged = bool(g.integers(0, 2))
    cfg = BASE.scaled(name=f"rand{seed}", L=int(g.integers(1, 4)), H=int(g.integers(1, 4)), d=d, T=T, r=r,
                      n_agents=4, paged=paged, page=int(g.choice([8, 16, 32, 64])), outliers=int(g.integers(0, 3)),
                      theta=float(g.choice([10000.0, 500000.0])), seed=seed)
    n_cov = int(g.choice([T, T, g.integers(0, T + 1)]))
    shift = int(g.choice([0, g.integers(-600, 600)]))
    pairing = int(g.choice([kvc.KVC_ROPE_HALF, kvc.KVC_ROPE_HALF, kvc.KVC_ROPE_INTERLEAVED]))
    bdt = torch.bfloat16 if g.integers(0, 4) == 0 else torch.float32
    return cfg, n_cov, shift, pairing, bdt


def _opair(pairing):
    return orc.ROPE_HALF if pairing == kvc.KVC_ROPE_HALF else orc.ROPE_INTERLEAVED


@pytest.mark.parametrize("seed", range(28))
def test_apply_random_shape(seed):
    cfg, n_cov, shift, pairing, bdt = _draw(seed)
    src_cpu = hp.make_cache(cfg)
    if n_cov:
        st_cpu = hp.make_state(cfg, 1 + seed % 3, n_cov=n_cov, basis_dtype=bdt)
    else:
        full = hp.make_state(cfg, 1, basis_dtype=bdt)
        st_cpu = kvc.State(None, None, full.basis_k, full.basis_v, n_cov=0)
    src = hp.to_dev(src_cpu, DEV)
    dst = hp.empty_dst(src_cpu, cfg, DEV, fill=-3.0)
    kvc.kvc_apply(src, hp.state_to_dev(st_cpu, DEV), shift, kvc.Rope(cfg.theta, pairing), dst)
    torch.cuda.synchronize()
    osrc = hp.oracle_cache(src_cpu)
    odst = osrc.empty_like(page_table=None if dst.page_table is None else dst.page_table.cpu().numpy())
    odst, ref_k, ref_v = orc.apply(osrc, hp.oracle_state(st_cpu), shift, hp.inv_freq(cfg), dst=odst,
                                   pairing=_opair(pairing), want_ref=True)
    gk, gv = hp.logical_bits(dst, "k"), hp.logical_bits(dst, "v")
    rk, rv = hp.tol_ratio(gk, ref_k), hp.tol_ratio(gv, ref_v)
    assert rk <= 1.0 and rv <= 1.0, (cfg, n_cov, shift, pairing, rk, rv)
    assert hp.ulp_mismatch_fraction(gk, hp.logical_bits(odst, "k")) < 1e-2
    assert hp.ulp_mismatch_fraction(gv, hp.logical_bits(odst, "v")) < 1e-2
    # rows behind the covered prefix: values pass through bit for bit
    assert np.array_equal(gv[:, :, n_cov:], hp.logical_bits(src_cpu, "v")[:, :, n_cov:])
    assert torch.equal(src.k.cpu(), src_cpu.k) and torch.equal(src.v.cpu(), src_cpu.v)
    if dst.page_table is not None:
        fill = torch.tensor(-3.0, dtype=torch.bfloat16)
        mapped = set(int(p) for p in dst.page_table.cpu())
        for p in range(dst.P):
            if p not in mapped:
                assert torch.all(dst.k[:, p].cpu() == fill) and torch.all(dst.v[:, p].cpu() == fill)
        tail = cfg.T % cfg.page
        if tail:
            last = int(dst.page_table[-1])
            assert torch.all(dst.k[:, last, :, tail:].cpu() == fill) and torch.all(dst.v[:, last, :, tail:].cpu() == fill)


@pytest.mark.parametrize("seed", range(100, 116))
def test_project_random_shape(seed):
    cfg, n_cov, shift, pairing, bdt = _draw(seed)
    n_cov = max(n_cov, 1)
    f = hp.inv_freq(cfg)
    src_cpu = hp.make_cache(cfg)
    true = hp.make_state(cfg, 1)
    nk = wl.noise((cfg.L, cfg.H, cfg.T, cfg.d), cfg.seed, 2).numpy()
    nv = wl.noise((cfg.L, cfg.H, cfg.T, cfg.d), cfg.seed, 3).numpy()
    osrc = hp.oracle_cache(src_cpu)
    otgt = orc.make_target(osrc, hp.oracle_state(true), shift, f, nk, nv, cfg.sigma, pairing=_opair(pairing))
    as_t = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
    if cfg.paged:
        tgt_cpu = kvc.Cache(as_t(otgt.k), as_t(otgt.v), T=cfg.T, page_table=src_cpu.page_table)
    else:
        tgt_cpu = kvc.Cache(as_t(otgt.k), as_t(otgt.v))
    other = hp.make_state(cfg, 3, basis_dtype=bdt)
    bk, bv = other.basis_k.float().numpy(), other.basis_v.float().numpy()
    ost, _ = orc.state_update(osrc, otgt, shift, f, mode=orc.PROJECT, n_cov=n_cov, basis_k=bk, basis_v=bv,
                              pairing=_opair(pairing))
    st = kvc.State(torch.full((cfg.L, cfg.H, n_cov, cfg.r), 7.0, device=DEV),
                   torch.full((cfg.L, cfg.H, n_cov, cfg.r), 7.0, device=DEV),
                   other.basis_k.to(DEV), other.basis_v.to(DEV), n_cov=n_cov)
    kvc.kvc_state_update(hp.to_dev(src_cpu, DEV), hp.to_dev(tgt_cpu, DEV), shift, kvc.Rope(cfg.theta, pairing), st,
                         kvc.KVC_PROJECT)
    torch.cuda.synchronize()
    worst = 0.0
    for l in range(cfg.L):
        for h in range(cfg.H):
            for which, got, ref, bs in (("k", st.coeff_k, ost.coeff_k, bk), ("v", st.coeff_v, ost.coeff_v, bv)):
                dl = orc.deviation(osrc.get_bits(which, l, h), otgt.get_bits(which, l, h), shift, f, which == "k",
                                   pairing=_opair(pairing))[:n_cov]
                bn = np.linalg.norm(bs[l, h].astype(np.float64), axis=1)[None, :]
                dn = np.linalg.norm(dl, axis=1)[:, None]
                sn = np.linalg.norm(orc.bf16_to_f64(osrc.get_bits(which, l, h)), axis=1)[:n_cov, None]
                tn = np.linalg.norm(orc.bf16_to_f64(otgt.get_bits(which, l, h)), axis=1)[:n_cov, None]
                # product rounding of the split-precision contraction; float32 rotation and
                # cancellation in tgt - Rot(src), relative to the inputs' size
                tol = 2.0 ** -12 * dn * bn + 2.0 ** -18 * (sn + tn) * bn + 1e-6
                err = np.abs(got[l, h].cpu().numpy().astype(np.float64) - ref[l, h].astype(np.float64))
                worst = max(worst, float(np.max(err / tol)))
    assert worst <= 1.0, (cfg, n_cov, shift, pairing, worst)


@pytest.mark.parametrize("seed", range(200, 212))
def test_chain_random_shape(seed):
    """kvc_chain against the oracle's chain at every hop; kvc_chain_fused equal to kvc_chain bit for bit
    (whether the fused kernel serves the shape or the call runs hop by hop)."""
    cfg, _, _, pairing, _ = _draw(seed)
    g = np.random.default_rng(88000 + seed)
    n = int(g.integers(2, 6))
    cfg = cfg.scaled(n_agents=n)
    pl = [int(x) for x in g.integers(0, 700, size=n)]
    states_cpu = []
    for a in range(1, n):
        kind = int(g.integers(0, 6))
        if kind == 0:
            states_cpu.append(kvc.State.empty())
            continue
        r = int(g.choice([4, 8, 16, 32, 48, 64, cfg.r]))
        n_cov = cfg.T if kind < 4 else int(g.integers(1, cfg.T + 1))
        bdt = torch.bfloat16 if kind == 3 else torch.float32
        states_cpu.append(hp.make_state(cfg, a, n_cov=n_cov, r=r, basis_dtype=bdt))
    rope = kvc.Rope(cfg.theta, pairing)
    src_cpu = hp.make_cache(cfg)
    src = hp.to_dev(src_cpu, DEV)
    states = [hp.state_to_dev(s, DEV) for s in states_cpu]
    ref = [hp.empty_dst(src_cpu, cfg, DEV, table_tag=60 + a, fill=2.0) for a in range(1, n)]
    got = [kvc.Cache(torch.full_like(o.k, 2.0), torch.full_like(o.v, 2.0), T=o.T if o.page_table is not None else None,
                     page_table=o.page_table) for o in ref]
    kvc.kvc_chain(src, pl, states, rope, ref)
    ws = torch.empty(max(kvc.kvc_chain_workspace_bytes(src, n), 128), dtype=torch.uint8, device=DEV)
    kvc.kvc_chain_fused(src, pl, states, rope, got, ws)
    torch.cuda.synchronize()
    for a, (x, y) in enumerate(zip(got, ref)):
        assert torch.equal(x.k, y.k) and torch.equal(x.v, y.v), (cfg, pl, a + 1)
    tables = [None if o.page_table is None else o.page_table.cpu().numpy() for o in ref]
    out, refs = orc.chain(hp.oracle_cache(src_cpu), pl, [hp.oracle_state(s) for s in states_cpu], hp.inv_freq(cfg),
                          dst_tables=tables, pairing=_opair(pairing), want_ref=True)
    for a in range(1, n):
        # strict parity of every hop from oracle-identical inputs: hop 1 reads agent 0, a later hop is run
        # once more from the ORACLE's materialised cache of the agent before (oracle -> library only)
        rk, rv = refs[a - 1]
        if a == 1:
            dst = ref[0]
        else:
            o_src = out[a - 2]
            as_t = lambda x: torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).to(DEV)
            hop_src = kvc.Cache(as_t(o_src.k), as_t(o_src.v), T=cfg.T if cfg.paged else None,
                                page_table=None if not cfg.paged else torch.from_numpy(o_src.page_table).to(DEV))
            dst = hp.empty_dst(src_cpu, cfg, DEV, table_tag=60 + a, fill=2.0)
            kvc.kvc_apply(hop_src, states[a - 1], pl[a] - pl[a - 1], rope, dst)
            torch.cuda.synchronize()
        assert hp.tol_ratio(hp.logical_bits(dst, "k"), rk) <= 1.0, (cfg, pl, a)
        assert hp.tol_ratio(hp.logical_bits(dst, "v"), rv) <= 1.0, (cfg, pl, a)
        # end to end the two chains stay together: a rare one-ulp difference at a hop moves the next
        # hop's input by one bf16 step, so this bar is statistical
        for which, r_ in (("k", rk), ("v", rv)):
            got_f = orc.bf16_to_f64(hp.logical_bits(ref[a - 1], which))
            bad = np.abs(got_f - r_) > hp.BF16_REL * np.abs(r_) + hp.BF16_ABS
            assert bad.mean() < 2e-3, (cfg, pl, a, which)


@pytest.mark.parametrize("mode", ["fit", "fit_fast"])
@pytest.mark.parametrize("seed", range(300, 310))
def test_fit_random_shape(seed, mode):
    """Both fit modes on drawn shapes (lengths below and above the rank and the head dimension, partial
    coverage, pages, shifts): the oracle's eigenvalues, orthonormal rows where the eigenvalue is not zero,
    zero rows beyond the number of covered tokens, a residual at the tail energy (Eckart-Young), and
    coefficients that are the projection of the deviation onto the library's own basis."""
    cfg, n_cov, shift, pairing, _ = _draw(seed)
    g = np.random.default_rng(99000 + seed)
    r_fit = int(g.choice([1, 4, 8, 16, 32])) if mode == "fit_fast" else int(g.choice([1, 4, 8, 16, 32, 33, 64]))
    r_fit = min(r_fit, cfg.d)
    n_cov = max(n_cov, 1)
    kmode = kvc.KVC_FIT if mode == "fit" else kvc.KVC_FIT_FAST
    f = hp.inv_freq(cfg)
    src_cpu = hp.make_cache(cfg)
    true = hp.make_state(cfg, 1, r=min(cfg.r, 8))
    nk = wl.noise((cfg.L, cfg.H, cfg.T, cfg.d), cfg.seed, 2).numpy()
    nv = wl.noise((cfg.L, cfg.H, cfg.T, cfg.d), cfg.seed, 3).numpy()
    osrc = hp.oracle_cache(src_cpu)
    otgt = orc.make_target(osrc, hp.oracle_state(true), shift, f, nk, nv, cfg.sigma, pairing=_opair(pairing))
    as_t = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
    if cfg.paged:
        tgt_cpu = kvc.Cache(as_t(otgt.k), as_t(otgt.v), T=cfg.T, page_table=src_cpu.page_table)
    else:
        tgt_cpu = kvc.Cache(as_t(otgt.k), as_t(otgt.v))
    L, H, d = cfg.L, cfg.H, cfg.d
    tgt = hp.to_dev(tgt_cpu, DEV)
    st = kvc.State(torch.full((L, H, n_cov, r_fit), 5.0, device=DEV), torch.full((L, H, n_cov, r_fit), 5.0, device=DEV),
                   torch.full((L, H, r_fit, d), 3.0, device=DEV), torch.full((L, H, r_fit, d), 3.0, device=DEV), n_cov=n_cov)
    ws = torch.zeros(kvc.kvc_workspace_bytes(tgt, st, kmode), dtype=torch.uint8, device=DEV)
    kvc.kvc_state_update(hp.to_dev(src_cpu, DEV), tgt, shift, kvc.Rope(cfg.theta, pairing), st, kmode, workspace=ws)
    torch.cuda.synchronize()
    m = L * H * 2
    ev = ws.view(torch.float32)[2 * m * d * d: 2 * m * d * d + m * d].cpu().numpy().astype(np.float64).reshape(L, H, 2, d)
    for l in range(L):
        for h in range(H):
            for i, (which, B_t, c_t) in enumerate((("k", st.basis_k, st.coeff_k), ("v", st.basis_v, st.coeff_v))):
                dl = orc.deviation(osrc.get_bits(which, l, h), otgt.get_bits(which, l, h), shift, f, which == "k",
                                   pairing=_opair(pairing))[:n_cov]
                w = np.sort(np.linalg.eigvalsh(orc.gram(dl)))[::-1]
                w = np.maximum(w, 0.0)
                B = B_t[l, h].cpu().numpy().astype(np.float64)
                c = c_t[l, h].cpu().numpy().astype(np.float64)
                what = (cfg, n_cov, shift, r_fit, l, h, which)
                if mode == "fit":
                    assert np.max(np.abs(ev[l, h, i] - w)) <= 1e-4 * w[0] + 1e-12, what
                live = min(r_fit, n_cov, d)
                assert np.all(B[live:] == 0), what                       # more rank asked for than rows exist
                Gb = B[:live] @ B[:live].T
                nz = np.diag(Gb) > 0.5                                   # rows of eigenvalue zero may be zero
                assert np.max(np.abs(Gb[np.ix_(nz, nz)] - np.eye(int(nz.sum())))) <= 1e-4, what
                assert np.all(w[:live][~nz] <= 1e-5 * w[0] + 1e-12), what
                res = float(np.sum((dl - c @ B) ** 2))
                tail = float(np.sum(w[r_fit:]))
                assert res <= 1.001 * tail + 8 * r_fit * 1.2e-6 * w[0] + 1e-9 * float(np.sum(w)) + 1e-9, what + (res, tail)
                bn = np.linalg.norm(B, axis=1)[None, :]
                dn = np.linalg.norm(dl, axis=1)[:, None]
                sn = np.linalg.norm(orc.bf16_to_f64(osrc.get_bits(which, l, h)), axis=1)[:n_cov, None]
                tn = np.linalg.norm(orc.bf16_to_f64(otgt.get_bits(which, l, h)), axis=1)[:n_cov, None]
                tol = 2.0 ** -12 * dn * bn + 2.0 ** -18 * (sn + tn) * bn + 1e-6
                assert np.max(np.abs(c - dl @ B.T) / tol) <= 1.0, what


@pytest.mark.parametrize("seed", range(400, 414))
def test_apply_segmented_random_shape(seed):
    """kvc_apply_segmented on drawn shapes with one to five drawn segments (boundaries anywhere, shifts of
    either sign or zero, both coordinate conventions) against the oracle's per-token-shift apply."""
    cfg, n_cov, _, _, bdt = _draw(seed)
    g = np.random.default_rng(55000 + seed)
    n_seg = int(g.integers(1, min(5, cfg.T) + 1))
    t_begin = [0] + sorted(int(x) for x in g.choice(np.arange(1, max(cfg.T, 2)), size=n_seg - 1, replace=False)) if cfg.T > 1 else [0]
    shift = [int(g.choice([0, g.integers(-600, 600)])) for _ in t_begin]
    coords = int(g.choice([kvc.KVC_COORDS_TARGET, kvc.KVC_COORDS_SOURCE]))
    n_cov = max(n_cov, 1)
    s_tok = orc.segment_shifts(cfg.T, t_begin, shift)
    f = hp.inv_freq(cfg)
    src_cpu = hp.make_cache(cfg)
    st_cpu = hp.make_state(cfg, 1, n_cov=n_cov, basis_dtype=bdt)
    dst = hp.empty_dst(src_cpu, cfg, DEV, fill=-3.0)
    kvc.kvc_apply_segmented(hp.to_dev(src_cpu, DEV), hp.state_to_dev(st_cpu, DEV), kvc.Segments(t_begin, shift, coords),
                            kvc.Rope(cfg.theta), dst)
    torch.cuda.synchronize()
    osrc, ost = hp.oracle_cache(src_cpu), hp.oracle_state(st_cpu)
    for which in ("k", "v"):
        got = hp.logical_bits(dst, which)
        for l in range(cfg.L):
            for h in range(cfg.H):
                c = (ost.coeff_k if which == "k" else ost.coeff_v)[l, h]
                b = (ost.basis_k if which == "k" else ost.basis_v)[l, h]
                ref, exp = orc.apply_slab_tokens(osrc.get_bits(which, l, h), c, b, s_tok, f, n_cov, which == "k", coords=coords)
                what = (cfg, n_cov, t_begin, shift, coords, which, l, h)
                assert hp.tol_ratio(got[l, h], ref) <= 1.0, what
                assert hp.ulp_mismatch_fraction(got[l, h], exp) < 1e-2, what
                keep = (s_tok == 0) & (np.arange(cfg.T) >= n_cov) if which == "k" else (np.arange(cfg.T) >= n_cov)
                assert np.array_equal(got[l, h][keep], osrc.get_bits(which, l, h)[keep]), what


@pytest.mark.parametrize("seed", range(500, 512))
def test_apply_multi_random_shape(seed):
    """kvc_apply_multi (Eq. 8, token-wise weights) on drawn shapes: one to five anchors of drawn ranks
    (multiples of 4 up to 64) and coverages, weighted or with unit weights, against the oracle."""
    cfg, _, shift, _, _ = _draw(seed)
    cfg = cfg.scaled(d=128)
    g = np.random.default_rng(66000 + seed)
    V = int(g.integers(1, 6))
    ranks = [int(g.choice([4, 8, 16, 20, 32, 48, 64])) for _ in range(V)]
    n_covs = [cfg.T if g.integers(0, 2) else int(g.integers(1, cfg.T + 1)) for _ in range(V)]
    anchors = [hp.make_state(cfg, hop=v + 1, r=r, n_cov=n) for v, (r, n) in enumerate(zip(ranks, n_covs))]
    src_cpu = hp.make_cache(cfg)
    wk = wv = None
    if g.integers(0, 3) > 0:
        tp = kvc.kvc_multi_tpad(cfg.T)

        def weights(tag):
            w = wl.noise((V, cfg.T), cfg.seed, 300 + tag, "cpu").abs() + 0.05
            w = w / w.sum(dim=0, keepdim=True)
            out = torch.zeros(V, tp, dtype=torch.float32)
            out[:, :cfg.T] = w
            return out
        wk, wv = weights(0), weights(1)
    src = hp.to_dev(src_cpu, DEV)
    dst = hp.empty_dst(src_cpu, cfg, DEV, fill=-7.0)
    dev_anchors = [hp.state_to_dev(a, DEV) for a in anchors]
    ws = torch.empty(max(kvc.kvc_multi_workspace_bytes(src, dev_anchors), 128), dtype=torch.uint8, device=DEV)
    mv = lambda t: None if t is None else t.to(DEV)
    kvc.kvc_apply_multi(src, dev_anchors, mv(wk), mv(wv), shift, kvc.Rope(cfg.theta), dst, ws)
    torch.cuda.synchronize()
    osrc = hp.oracle_cache(src_cpu)
    inv = hp.inv_freq(cfg)
    for which, w in (("k", wk), ("v", wv)):
        got = hp.logical_bits(dst, which)
        for l in range(cfg.L):
            for h in range(cfg.H):
                ref, out = orc.apply_multi_slab(
                    osrc.get_bits(which, l, h), None if w is None else w.numpy()[:, :cfg.T],
                    [getattr(a, "coeff_" + which)[l, h].numpy() for a in anchors],
                    [getattr(a, "basis_" + which)[l, h].to(torch.float32).numpy() for a in anchors],
                    n_covs, shift, inv, which == "k", orc.ROPE_HALF)
                what = (cfg, ranks, n_covs, shift, which, l, h)
                assert hp.tol_ratio(got[l, h], ref) <= 1.0, what
                assert hp.ulp_mismatch_fraction(got[l, h], out) < 2e-2, what


@pytest.mark.parametrize("seed", range(600, 608))
def test_apply_batch_random_items(seed):
    """kvc_apply_batch over three to nine items whose shapes are drawn independently (rank,
    layers, heads, length, layout, coverage, shift differ from item to item; some states are empty): every
    item equals its own kvc_apply bit for bit and meets the oracle."""
    g = np.random.default_rng(44000 + seed)
    n = int(g.integers(3, 10))
    rope_theta = float(g.choice([10000.0, 500000.0]))
    rope = kvc.Rope(rope_theta)
    d_batch = int(g.choice([64, 128, 128]))
    items, singles, oracles = [], [], []
    for i in range(n):
        cfg, n_cov, shift, _, bdt = _draw(1000 * seed + i)
        cfg = cfg.scaled(theta=rope_theta, d=d_batch)         # the items of a launch share head_dim
        src_cpu = hp.make_cache(cfg)
        kind = int(g.integers(0, 5))
        if kind == 0 or n_cov == 0:
            st_cpu = kvc.State.empty()
        else:
            st_cpu = hp.make_state(cfg, 1 + i % 3, n_cov=n_cov, basis_dtype=bdt)
        src, st = hp.to_dev(src_cpu, DEV), hp.state_to_dev(st_cpu, DEV)
        dst = hp.empty_dst(src_cpu, cfg, DEV, fill=1.0)
        one = hp.empty_dst(src_cpu, cfg, DEV, fill=1.0)
        items.append(kvc.Item(src, dst, st, shift))
        singles.append((src, st, shift, one))
        oracles.append((cfg, src_cpu, st_cpu, shift))
    nb = kvc.kvc_batch_workspace_bytes(len(items))
    ws = torch.empty(nb, dtype=torch.uint8, device=DEV)
    staging = torch.empty(nb, dtype=torch.uint8).pin_memory()
    kvc.kvc_apply_batch(items, rope, ws, staging)
    batch_path = kvc.kvc_last_path()
    single_path = []
    for (src, st, shift, one) in singles:
        kvc.kvc_apply(src, st, shift, rope, one)
        single_path.append(kvc.kvc_last_path())
    torch.cuda.synchronize()
    # every item runs on the kernel family it would get alone (a launch splits between the two), so the bits agree
    assert batch_path == (kvc.KVC_PATH_MIXED if len(set(single_path)) == 2 else single_path[0])
    for i, (it, (_, _, _, one), (cfg, src_cpu, st_cpu, shift)) in enumerate(zip(items, singles, oracles)):
        assert torch.equal(it.dst.k, one.k) and torch.equal(it.dst.v, one.v), (cfg, shift)
        osrc = hp.oracle_cache(src_cpu)
        odst = osrc.empty_like(page_table=None if it.dst.page_table is None else it.dst.page_table.cpu().numpy())
        odst, ref_k, ref_v = orc.apply(osrc, hp.oracle_state(st_cpu), shift, hp.inv_freq(cfg), dst=odst, want_ref=True)
        assert hp.tol_ratio(hp.logical_bits(it.dst, "k"), ref_k) <= 1.0, (cfg, shift)
        assert hp.tol_ratio(hp.logical_bits(it.dst, "v"), ref_v) <= 1.0, (cfg, shift)


@pytest.mark.parametrize("seed", range(700, 712))
def test_grouped_apply_and_gate_random_shape(seed):
    """Per-layer states (D = H d, Sec. 3.1) on drawn shapes through kvc_apply, and the gate distance (Eq. 9)
    of the same source against drawn per-head anchors at a drawn comparison length."""
    cfg, n_cov, shift, pairing, bdt = _draw(seed)
    g = np.random.default_rng(33000 + seed)
    n_cov = max(n_cov, 1)
    one = cfg.scaled(H=1, d=cfg.H * cfg.d)
    r = min(cfg.r, 64)
    ck = wl.coefficients(cfg.L, 1, cfg.T, r, cfg.seed, 4, "cpu")[:, 0, :n_cov].contiguous()
    cv = wl.coefficients(cfg.L, 1, cfg.T, r, cfg.seed, 5, "cpu")[:, 0, :n_cov].contiguous()
    bk = wl.orthonormal_basis(cfg.L, 1, r, one.d, cfg.seed, 6, "cpu")[:, 0].contiguous().to(bdt)
    bv = wl.orthonormal_basis(cfg.L, 1, r, one.d, cfg.seed, 7, "cpu")[:, 0].contiguous().to(bdt)
    st = kvc.State(ck, cv, bk, bv, n_cov=n_cov, grouping=kvc.KVC_GROUP_LAYER)
    src_cpu = hp.make_cache(cfg)
    src = hp.to_dev(src_cpu, DEV)
    dst = hp.empty_dst(src_cpu, cfg, DEV, fill=3.0)
    kvc.kvc_apply(src, hp.state_to_dev(st, DEV), shift, kvc.Rope(cfg.theta, pairing), dst)
    torch.cuda.synchronize()
    f32 = lambda t: t.to(torch.float32).numpy()
    ost = orc.ungroup_state(f32(ck), f32(cv), f32(bk), f32(bv), cfg.H, n_cov=n_cov)
    osrc = hp.oracle_cache(src_cpu)
    odst = osrc.empty_like(page_table=None if dst.page_table is None else dst.page_table.cpu().numpy())
    odst, rk, rv = orc.apply(osrc, ost, shift, hp.inv_freq(cfg), dst=odst, pairing=_opair(pairing), want_ref=True)
    gk, gv = hp.logical_bits(dst, "k"), hp.logical_bits(dst, "v")
    assert hp.tol_ratio(gk, rk) <= 1.0 and hp.tol_ratio(gv, rv) <= 1.0, (cfg, n_cov, shift, pairing)
    assert hp.ulp_mismatch_fraction(gk, hp.logical_bits(odst, "k")) < 1e-2
    assert hp.ulp_mismatch_fraction(gv, hp.logical_bits(odst, "v")) < 1e-2
    # ---- gate distance against two per-head anchors
    anchors = [hp.make_state(cfg, hop=v + 1, basis_dtype=bdt if v else torch.float32) for v in range(2)]
    k = int(g.integers(1, cfg.T + 1))
    d2 = torch.full((2,), -1.0, dtype=torch.float64, device=DEV)
    kvc.kvc_gate_distance(src, [hp.state_to_dev(a, DEV) for a in anchors], k, d2)
    torch.cuda.synchronize()
    ref = []
    for a in anchors:
        c = a.coeff_v.numpy().astype(np.float64)
        b = a.basis_v.to(torch.float32).numpy().astype(np.float64)
        v_src = [np.concatenate([orc.bf16_to_f64(osrc.get_bits("v", l, h)) for h in range(cfg.H)], axis=1) for l in range(cfg.L)]
        v_anc = [np.concatenate([c[l, h] @ b[l, h] for h in range(cfg.H)], axis=1) for l in range(cfg.L)]
        ref.append(orc.gate_distance(v_src, v_anc, k))
    ref = np.array(ref)
    got = np.sqrt(d2.cpu().numpy())
    assert np.all(np.abs(got - ref) <= 1e-4 * ref + 1e-6), (cfg, k, got, ref)
