"""Multi-segment contexts (Eq. 1) and the two coordinate conventions of the correction (Eq. 12, App. A.2)
through kvc_apply_segmented / kvc_state_update_segmented, against the oracle's per-token-shift functions.

Three segments with different shifts (one of them zero), boundaries that fall neither on a page nor on a
tile, contiguous and paged caches, per-head and layer-grouped states.
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

CFG_C = wl.CONFIGS["llama8b_8k"].scaled(name="8b_small", L=2, H=2, T=700)
CFG_P = wl.CONFIGS["vlm_16k"].scaled(name="vlm_small", L=1, H=2, T=1003, image_spans=())
CFG_T = wl.CONFIGS["tiny"]
SEGS = {"8b_small": ([0, 133, 390], [37, 0, -211]), "vlm_small": ([0, 21, 530], [-5, 512, 64]), "tiny": ([0, 7, 100], [3, -2, 0]),
        # several segments inside one 16-token page, and one that ends inside the page the next begins in
        "vlm_short_segments": ([0, 5, 9, 40, 300], [3, -7, 0, 25, -100])}
CFG_PS = CFG_P.scaled(name="vlm_short_segments", T=403)
COORDS = [kvc.KVC_COORDS_TARGET, kvc.KVC_COORDS_SOURCE]


@pytest.fixture(autouse=True)
def _clean_status():
    kvc.kvc_status_reset()
    yield
    kvc.kvc_set_path(kvc.KVC_PATH_AUTO)
    assert kvc.kvc_status_poll() == 0


@pytest.mark.parametrize("path", [kvc.KVC_PATH_GENERIC, kvc.KVC_PATH_AUTO], ids=["generic", "auto"])
@pytest.mark.parametrize("coords", COORDS, ids=["target", "source"])
@pytest.mark.parametrize("cfg", [CFG_C, CFG_P, CFG_T], ids=lambda c: c.name)
def test_apply_segmented(cfg, coords, path):
    kvc.kvc_set_path(path)
    t_begin, shift = SEGS[cfg.name]
    s_tok = orc.segment_shifts(cfg.T, t_begin, shift)
    f = hp.inv_freq(cfg)
    src_cpu = hp.make_cache(cfg)
    n_cov = cfg.T - 45                              # the last rows are only re-aligned
    st_cpu = hp.make_state(cfg, 1, n_cov=n_cov)
    dst = hp.empty_dst(src_cpu, cfg, DEV)
    kvc.kvc_apply_segmented(hp.to_dev(src_cpu, DEV), hp.state_to_dev(st_cpu, DEV), kvc.Segments(t_begin, shift, coords),
                            kvc.Rope(cfg.theta), dst)
    torch.cuda.synchronize()
    assert kvc.kvc_last_path() == (kvc.KVC_PATH_TC if (path == kvc.KVC_PATH_AUTO and cfg.d == 128) else kvc.KVC_PATH_GENERIC)
    osrc, ost = hp.oracle_cache(src_cpu), hp.oracle_state(st_cpu)
    for which in ("k", "v"):
        got = hp.logical_bits(dst, which)
        for l in range(cfg.L):
            for h in range(cfg.H):
                c = (ost.coeff_k if which == "k" else ost.coeff_v)[l, h]
                b = (ost.basis_k if which == "k" else ost.basis_v)[l, h]
                ref, exp = orc.apply_slab_tokens(osrc.get_bits(which, l, h), c, b, s_tok, f, n_cov, which == "k", coords=coords)
                assert hp.tol_ratio(got[l, h], ref) <= 1.0, (which, l, h)
                assert hp.ulp_mismatch_fraction(got[l, h], exp) < 1e-2
                # rows that are neither covered nor shifted keep their bits
                keep = (s_tok == 0) & (np.arange(cfg.T) >= n_cov) if which == "k" else (np.arange(cfg.T) >= n_cov)
                assert np.array_equal(got[l, h][keep], osrc.get_bits(which, l, h)[keep])


@pytest.mark.parametrize("coords", COORDS, ids=["target", "source"])
@pytest.mark.parametrize("cfg,on_pages", [(CFG_C, False), (CFG_P, False), (CFG_P, True), (CFG_PS, False)],
                         ids=["8b_small", "vlm_small", "vlm_small-page-aligned", "vlm_short_segments"])
def test_project_and_fit_segmented(cfg, on_pages, coords):
    """PROJECT: coefficients of the per-token-shift deviation in a given basis.  FIT: the deviation is built
    exactly rank r in the chosen coordinates, so the fitted state reproduces the oracle's subspace and the
    update -> apply round trip gives back the target."""
    t_begin, shift = SEGS[cfg.name]
    if on_pages:                                   # boundaries on the 16-token page grid: tensor-core windows on a paged source
        t_begin = [0, 32, 528]
    s_tok = orc.segment_shifts(cfg.T, t_begin, shift)
    f = hp.inv_freq(cfg)
    segs = kvc.Segments(t_begin, shift, coords)
    rope = kvc.Rope(cfg.theta)
    src_cpu = hp.make_cache(cfg)
    true = hp.make_state(cfg, 1)
    osrc, otrue = hp.oracle_cache(src_cpu), hp.oracle_state(true)
    # the target: the oracle's segmented apply of the true state (+ noise), rounded to bf16
    tk, tv = np.zeros_like(hp.logical_bits(src_cpu, "k")), np.zeros_like(hp.logical_bits(src_cpu, "v"))
    nz = {w: wl.noise((cfg.L, cfg.H, cfg.T, cfg.d), cfg.seed, 2 + i).numpy() for i, w in enumerate(("k", "v"))}
    for which, out in (("k", tk), ("v", tv)):
        for l in range(cfg.L):
            for h in range(cfg.H):
                c = (otrue.coeff_k if which == "k" else otrue.coeff_v)[l, h]
                b = (otrue.basis_k if which == "k" else otrue.basis_v)[l, h]
                ref, _ = orc.apply_slab_tokens(osrc.get_bits(which, l, h), c, b, s_tok, f, cfg.T, which == "k", coords=coords)
                out[l, h] = orc.f64_to_bf16_bits(ref + cfg.sigma * nz[which][l, h])
    as_t = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
    tgt_cpu = kvc.Cache(as_t(tk), as_t(tv))                 # contiguous target, whatever the source's layout
    src, tgt = hp.to_dev(src_cpu, DEV), hp.to_dev(tgt_cpu, DEV)
    L, H, T, d, r = cfg.L, cfg.H, cfg.T, cfg.d, cfg.r
    # ---- PROJECT with a given basis
    given = hp.make_state(cfg, 2)
    st = kvc.State(torch.zeros(L, H, T, r, device=DEV), torch.zeros(L, H, T, r, device=DEV),
                   given.basis_k.to(DEV), given.basis_v.to(DEV))
    kvc.kvc_state_update_segmented(src, tgt, segs, rope, st, kvc.KVC_PROJECT)
    torch.cuda.synchronize()
    # a tensor-core launch per segment window, also where the boundaries of a paged cache are off the page grid
    # (the windows then start at the page's first row and the segments are launched from the last to the first)
    assert kvc.kvc_last_path() == (kvc.KVC_PATH_TC if cfg.d == 128 else kvc.KVC_PATH_GENERIC)
    deltas = {}
    for which, cf, bs in (("k", st.coeff_k, given.basis_k), ("v", st.coeff_v, given.basis_v)):
        for l in range(L):
            for h in range(H):
                sb = osrc.get_bits(which, l, h)
                tb = (tk if which == "k" else tv)[l, h]
                dl = orc.deviation_tokens(sb, tb, s_tok, f, which == "k", coords=coords)
                deltas[(which, l, h)] = dl
                B = bs[l, h].numpy().astype(np.float64)
                ref = orc.project(dl, B)
                got = cf[l, h].cpu().numpy().astype(np.float64)
                tol = 1e-5 * (np.linalg.norm(orc.bf16_to_f64(sb), axis=1) + np.linalg.norm(orc.bf16_to_f64(tb), axis=1))[:, None] + 1e-6
                assert np.max(np.abs(got - ref) / tol) <= 1.0, (which, l, h)
    # ---- FIT, then apply: the round trip
    for mode in (kvc.KVC_FIT, kvc.KVC_FIT_FAST):
        fit = kvc.State(torch.zeros(L, H, T, r, device=DEV), torch.zeros(L, H, T, r, device=DEV),
                        torch.zeros(L, H, r, d, device=DEV), torch.zeros(L, H, r, d, device=DEV))
        ws = torch.zeros(kvc.kvc_workspace_bytes(tgt, fit, mode), dtype=torch.uint8, device=DEV)
        kvc.kvc_state_update_segmented(src, tgt, segs, rope, fit, mode, workspace=ws)
        torch.cuda.synchronize()
        for which, Bt, ct in (("k", fit.basis_k, fit.coeff_k), ("v", fit.basis_v, fit.coeff_v)):
            for l in range(L):
                for h in range(H):
                    dl = deltas[(which, l, h)]
                    w = np.linalg.eigvalsh(orc.gram(dl))[::-1]
                    B = Bt[l, h].cpu().numpy().astype(np.float64)
                    c = ct[l, h].cpu().numpy().astype(np.float64)
                    assert np.max(np.abs(B @ B.T - np.eye(r))) <= 1e-4
                    res = float(np.sum((dl - c @ B) ** 2))
                    assert res <= 1.001 * float(np.sum(w[r:])) + 1e-6 * float(np.sum(w)), (mode, which, l, h)
        dst = kvc.Cache(torch.zeros_like(tgt.k), torch.zeros_like(tgt.v))
        kvc.kvc_apply_segmented(src, fit, segs, rope, dst)
        torch.cuda.synchronize()
        for which, want_bits in (("k", tk), ("v", tv)):
            got = orc.bf16_to_f64(hp.logical_bits(dst, which))
            want = orc.bf16_to_f64(want_bits)
            assert np.mean(np.abs(got - want) > 2.0 ** -6 * np.abs(want) + 0.02) < 1e-3


def test_one_segment_is_the_plain_call_and_source_coordinates_are_the_realigned_basis():
    cfg = CFG_C.scaled(T=333)
    rope = kvc.Rope(cfg.theta)
    src_cpu = hp.make_cache(cfg)
    st = hp.state_to_dev(hp.make_state(cfg, 1), DEV)
    src = hp.to_dev(src_cpu, DEV)
    shift = 77
    kvc.kvc_set_path(kvc.KVC_PATH_GENERIC)
    a, b = hp.empty_dst(src_cpu, cfg, DEV), hp.empty_dst(src_cpu, cfg, DEV)
    kvc.kvc_apply(src, st, shift, rope, a)
    kvc.kvc_apply_segmented(src, st, kvc.Segments([0], [shift]), rope, b)
    torch.cuda.synchronize()
    assert torch.equal(a.k, b.k) and torch.equal(a.v, b.v)            # same kernel, same tables: same bits
    # SOURCE coordinates with one shift = TARGET coordinates with the key basis rotated by that shift (App. A.2)
    re = kvc.kvc_state_realign(st, shift, rope)
    c, d_ = hp.empty_dst(src_cpu, cfg, DEV), hp.empty_dst(src_cpu, cfg, DEV)
    kvc.kvc_apply_segmented(src, st, kvc.Segments([0], [shift], kvc.KVC_COORDS_SOURCE), rope, c)
    kvc.kvc_apply(src, re, shift, rope, d_)
    torch.cuda.synchronize()
    diff = (c.k.float() - d_.k.float()).abs()
    assert float((diff > 2.0 ** -7 * d_.k.float().abs() + 1e-3).float().mean()) == 0.0
    assert torch.equal(c.v, d_.v)


def test_segment_argument_errors():
    cfg = CFG_T
    src_cpu = hp.make_cache(cfg)
    src, st = hp.to_dev(src_cpu, DEV), hp.state_to_dev(hp.make_state(cfg, 1), DEV)
    dst = hp.empty_dst(src_cpu, cfg, DEV)
    rope = kvc.Rope(cfg.theta)
    for bad in (kvc.Segments([5], [1]), kvc.Segments([0, 90, 40], [1, 2, 3]), kvc.Segments([0, cfg.T + 1], [1, 2]),
                kvc.Segments([0], [1], coords=5), kvc.Segments(list(range(17)), [0] * 17)):
        with pytest.raises(kvc.KvcError) as e:
            kvc.kvc_apply_segmented(src, st, bad, rope, dst)
        assert e.value.code == kvc.KVC_E_INVALID_ARG
    # the update passes with segment tables are CUDA-core kernels: forcing the tensor-core family is refused
    kvc.kvc_set_path(kvc.KVC_PATH_TC)
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_state_update_segmented(src, src, kvc.Segments([0, 9], [1, 2]), rope, st, kvc.KVC_PROJECT)
    assert e.value.code == kvc.KVC_E_UNSUPPORTED


def test_grouped_state_with_segments():
    """A layer-grouped state (D = H d) through the segmented calls: apply against the oracle's expanded
    per-head form, and FIT of a deviation of rank r across the heads (SOURCE coordinates)."""
    from test_gpu_grouped import _grouped_state, _oracle_state
    cfg = wl.CONFIGS["llama8b_8k"].scaled(name="8b_small", L=1, H=4, T=520, r=16)
    t_begin, shift = [0, 133, 390], [37, 0, -211]
    s_tok = orc.segment_shifts(cfg.T, t_begin, shift)
    f = hp.inv_freq(cfg)
    rope = kvc.Rope(cfg.theta)
    src_cpu = hp.make_cache(cfg)
    gst = _grouped_state(cfg, 1)
    ost = _oracle_state(cfg, gst)
    osrc = hp.oracle_cache(src_cpu)
    src = hp.to_dev(src_cpu, DEV)
    coords = kvc.KVC_COORDS_SOURCE
    segs = kvc.Segments(t_begin, shift, coords)
    dst = hp.empty_dst(src_cpu, cfg, DEV)
    kvc.kvc_apply_segmented(src, hp.state_to_dev(gst, DEV), segs, rope, dst)
    torch.cuda.synchronize()
    refs = {}
    for which in ("k", "v"):
        got = hp.logical_bits(dst, which)
        for h in range(cfg.H):
            c = (ost.coeff_k if which == "k" else ost.coeff_v)[0, h]
            b = (ost.basis_k if which == "k" else ost.basis_v)[0, h]
            ref, exp = orc.apply_slab_tokens(osrc.get_bits(which, 0, h), c, b, s_tok, f, cfg.T, which == "k", coords=coords)
            refs[(which, h)] = ref
            assert hp.tol_ratio(got[0, h], ref) <= 1.0
    # the corrected cache (its bf16 form) as the target of a grouped FIT in the same coordinates
    tgt = kvc.Cache(dst.k.clone(), dst.v.clone())
    L, H, T, d, r = cfg.L, cfg.H, cfg.T, cfg.d, cfg.r
    fit = kvc.State(torch.zeros(L, T, r, device=DEV), torch.zeros(L, T, r, device=DEV),
                    torch.zeros(L, r, H * d, device=DEV), torch.zeros(L, r, H * d, device=DEV), grouping=kvc.KVC_GROUP_LAYER)
    ws = torch.zeros(kvc.kvc_workspace_bytes(tgt, fit, kvc.KVC_FIT), dtype=torch.uint8, device=DEV)
    kvc.kvc_state_update_segmented(src, tgt, segs, rope, fit, kvc.KVC_FIT, workspace=ws)
    torch.cuda.synchronize()
    assert bool((kvc.kvc_group_fit_solver(tgt, ws) == 0).all())
    for i, (which, Bt, Bo) in enumerate((("k", fit.basis_k, gst.basis_k), ("v", fit.basis_v, gst.basis_v))):
        B = Bt[0].cpu().numpy().astype(np.float64)
        Btrue = Bo[0].numpy().astype(np.float64)
        assert np.max(np.abs(B @ B.T - np.eye(r))) <= 1e-4
        assert np.linalg.norm(B.T @ B - Btrue.T @ Btrue) <= 2e-2          # the rows span the true basis' space


# ---------------------------------------------------------------------------------------------------------
# The same multi-segment context as ONE launch of kvc_apply_batch: an item per segment over the same
# caches, each with its token range and its own shift.
# ---------------------------------------------------------------------------------------------------------
ITEM_SEGS = {"8b_small": ([0, 133, 390], [37, 0, -211]),      # contiguous: boundaries anywhere
             "vlm_small": ([0, 32, 528], [-5, 512, 64])}      # paged: boundaries on 16-token pages


@pytest.mark.parametrize("path", [kvc.KVC_PATH_GENERIC, kvc.KVC_PATH_AUTO], ids=["generic", "auto"])
@pytest.mark.parametrize("cfg", [CFG_C, CFG_P], ids=lambda c: c.name)
def test_batch_items_with_token_ranges(cfg, path):
    kvc.kvc_set_path(path)
    t_begin, shift = ITEM_SEGS[cfg.name]
    T = cfg.T
    t_stop = T - 29                                 # the last rows belong to no item: they keep the fill
    s_tok = orc.segment_shifts(T, t_begin, shift)
    f = hp.inv_freq(cfg)
    src_cpu = hp.make_cache(cfg)
    n_cov = t_begin[2] + 77                         # the coverage ends inside the last segment
    st_cpu = hp.make_state(cfg, 1, n_cov=n_cov)
    src, st = hp.to_dev(src_cpu, DEV), hp.state_to_dev(st_cpu, DEV)
    dst = hp.empty_dst(src_cpu, cfg, DEV, fill=1.0)
    ends = t_begin[1:] + [t_stop]
    items = [kvc.Item(src, dst, st, sh, tb, te) for tb, te, sh in zip(t_begin, ends, shift)]
    nb = kvc.kvc_batch_workspace_bytes(len(items))
    ws = torch.empty(nb, dtype=torch.uint8, device=DEV)
    staging = torch.empty(nb, dtype=torch.uint8).pin_memory()
    kvc.kvc_apply_batch(items, kvc.Rope(cfg.theta), ws, staging)
    torch.cuda.synchronize()
    assert kvc.kvc_last_path() == (kvc.KVC_PATH_TC if path == kvc.KVC_PATH_AUTO else kvc.KVC_PATH_GENERIC)
    osrc, ost = hp.oracle_cache(src_cpu), hp.oracle_state(st_cpu)
    one = orc.f64_to_bf16_bits(np.ones(1))[0]
    for which in ("k", "v"):
        got = hp.logical_bits(dst, which)
        for l in range(cfg.L):
            for h in range(cfg.H):
                c = (ost.coeff_k if which == "k" else ost.coeff_v)[l, h]
                b = (ost.basis_k if which == "k" else ost.basis_v)[l, h]
                ref, exp = orc.apply_slab_tokens(osrc.get_bits(which, l, h), c, b, s_tok, f, n_cov, which == "k")
                assert hp.tol_ratio(got[l, h][:t_stop], ref[:t_stop]) <= 1.0, (which, l, h)
                assert hp.ulp_mismatch_fraction(got[l, h][:t_stop], exp[:t_stop]) < 1e-2
                assert np.all(got[l, h][t_stop:] == one), "rows outside every item's range were written"


def test_batch_item_range_errors():
    cfg = CFG_P
    src_cpu = hp.make_cache(cfg)
    st = hp.state_to_dev(hp.make_state(cfg, 1), DEV)
    src = hp.to_dev(src_cpu, DEV)
    dst = hp.empty_dst(src_cpu, cfg, DEV)
    nb = kvc.kvc_batch_workspace_bytes(1)
    ws = torch.empty(nb, dtype=torch.uint8, device=DEV)
    staging = torch.empty(nb, dtype=torch.uint8).pin_memory()
    rope = kvc.Rope(cfg.theta)
    for tb, te, code in ((10, 5, kvc.KVC_E_INVALID_ARG), (0, cfg.T + 1, kvc.KVC_E_INVALID_ARG), (-16, 32, kvc.KVC_E_INVALID_ARG),
                         (8, 64, kvc.KVC_E_UNSUPPORTED)):        # a paged range must start on a page boundary
        with pytest.raises(kvc.KvcError) as e:
            kvc.kvc_apply_batch([kvc.Item(src, dst, st, 3, tb, te)], rope, ws, staging)
        assert e.value.code == code, (tb, te, str(e.value))
