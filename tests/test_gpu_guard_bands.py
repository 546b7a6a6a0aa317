"""Guard bands: every output of the library sits inside a larger allocation whose margins hold a sentinel;
after the call the margins must be untouched, whatever kernel family ran.  (The stand-in on this pool for a
memory checker: an out-of-range store of a kernel lands in a margin or in a neighbouring output's margin.)
Ragged lengths are used on purpose: the last tile of every slab is partial."""
import numpy as np
import pytest
import torch

import paper_2609_34060_b200 as kvc
from paper_2609_34060_b200 import workloads as wl

import helpers as hp

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
MARGIN = 4096          # elements on either side
PATHS = [kvc.KVC_PATH_GENERIC, kvc.KVC_PATH_AUTO]
PATH_IDS = ["generic", "auto"]


def _guarded(shape, dtype, fill):
    """A tensor of `shape` carved out of the middle of a sentinel-filled allocation (16-byte aligned)."""
    n = int(np.prod(shape))
    buf = torch.full((n + 2 * MARGIN,), fill, dtype=dtype, device=DEV)
    return buf, buf[MARGIN:MARGIN + n].view(shape)


def _intact(buf, n, fill):
    lo, hi = buf[:MARGIN], buf[MARGIN + n:]
    f = torch.tensor(fill, dtype=buf.dtype, device=DEV)
    return bool((lo == f).all()) and bool((hi == f).all())


@pytest.fixture(autouse=True)
def _clean_status():
    kvc.kvc_status_reset()
    yield
    kvc.kvc_set_path(kvc.KVC_PATH_AUTO)
    assert kvc.kvc_status_poll() == 0


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
@pytest.mark.parametrize("T", [129, 700, 1003])
def test_apply_chain_and_update_stay_inside_their_outputs(path, T):
    cfg = wl.CONFIGS["llama8b_8k"].scaled(name="guard", L=2, H=2, T=T, n_agents=3)
    L, H, d, r = cfg.L, cfg.H, cfg.d, cfg.r
    rope = kvc.Rope(cfg.theta)
    pl = wl.prefix_lengths(cfg)
    kvc.kvc_set_path(path)
    src = hp.to_dev(hp.make_cache(cfg), DEV)
    states = [hp.state_to_dev(hp.make_state(cfg, a), DEV) for a in (1, 2)]
    shape = (L, H, T, d)
    n = L * H * T * d
    outs, bufs = [], []
    for _ in range(2):
        bk, k = _guarded(shape, torch.bfloat16, 7.0)
        bv, v = _guarded(shape, torch.bfloat16, 7.0)
        outs.append(kvc.Cache(k, v))
        bufs += [bk, bv]
    kvc.kvc_chain(src, pl, states, rope, outs)
    torch.cuda.synchronize()
    assert all(_intact(b, n, 7.0) for b in bufs)
    # the fused chain writes the same outputs in one pass
    cws = torch.empty(max(kvc.kvc_chain_workspace_bytes(src, 3), 128), dtype=torch.uint8, device=DEV)
    kvc.kvc_chain_fused(src, pl, states, rope, outs, cws)
    torch.cuda.synchronize()
    assert all(_intact(b, n, 7.0) for b in bufs)
    # state update: coefficients, bases and the workspace are outputs
    for mode in (kvc.KVC_PROJECT, kvc.KVC_FIT, kvc.KVC_FIT_FAST):
        nc = L * H * T * r
        nb = L * H * r * d
        bck, ck = _guarded((L, H, T, r), torch.float32, -3.0)
        bcv, cv = _guarded((L, H, T, r), torch.float32, -3.0)
        bbk, bk_ = _guarded((L, H, r, d), torch.float32, -3.0)
        bbv, bv_ = _guarded((L, H, r, d), torch.float32, -3.0)
        bk_.copy_(states[0].basis_k)
        bv_.copy_(states[0].basis_v)
        st = kvc.State(ck, cv, bk_, bv_)
        need = kvc.kvc_workspace_bytes(outs[0], st, mode)
        bws = torch.full((need + 2 * MARGIN,), 0x5A, dtype=torch.uint8, device=DEV)
        off = (-bws.data_ptr() - MARGIN) % 256
        ws = bws[MARGIN + off: MARGIN + off + need]
        kvc.kvc_state_update(src, outs[0], pl[1] - pl[0], rope, st, mode, workspace=ws if need else None)
        torch.cuda.synchronize()
        assert _intact(bck, nc, -3.0) and _intact(bcv, nc, -3.0) and _intact(bbk, nb, -3.0) and _intact(bbv, nb, -3.0), mode
        assert bool((bws[:MARGIN + off] == 0x5A).all()) and bool((bws[MARGIN + off + need:] == 0x5A).all()), mode
        assert float(ck.abs().max()) != 3.0


def test_grouped_fit_and_segmented_calls_stay_inside_their_outputs():
    cfg = wl.CONFIGS["llama8b_8k"].scaled(name="guard_g", L=1, H=4, T=515, r=16)
    L, H, T, d, r = cfg.L, cfg.H, cfg.T, cfg.d, cfg.r
    rope = kvc.Rope(cfg.theta)
    src = hp.to_dev(hp.make_cache(cfg), DEV)
    tgt = hp.to_dev(hp.make_cache(cfg.scaled(seed=cfg.seed + 1)), DEV)
    bck, ck = _guarded((L, T, r), torch.float32, -3.0)
    bcv, cv = _guarded((L, T, r), torch.float32, -3.0)
    bbk, bk_ = _guarded((L, r, H * d), torch.float32, -3.0)
    bbv, bv_ = _guarded((L, r, H * d), torch.float32, -3.0)
    st = kvc.State(ck, cv, bk_, bv_, grouping=kvc.KVC_GROUP_LAYER)
    need = kvc.kvc_workspace_bytes(tgt, st, kvc.KVC_FIT)
    bws = torch.full((need + 2 * MARGIN,), 0x5A, dtype=torch.uint8, device=DEV)
    off = (-bws.data_ptr() - MARGIN) % 256
    ws = bws[MARGIN + off: MARGIN + off + need]
    for segs in (None, kvc.Segments([0, 100, 333], [5, 0, -40], kvc.KVC_COORDS_SOURCE)):
        if segs is None:
            kvc.kvc_state_update(src, tgt, 21, rope, st, kvc.KVC_FIT, workspace=ws)
        else:
            kvc.kvc_state_update_segmented(src, tgt, segs, rope, st, kvc.KVC_FIT, workspace=ws)
        torch.cuda.synchronize()
        kvc.kvc_status_reset()          # two unrelated Gaussian caches have no gap: the flag is expected here
        assert _intact(bck, L * T * r, -3.0) and _intact(bcv, L * T * r, -3.0)
        assert _intact(bbk, L * r * H * d, -3.0) and _intact(bbv, L * r * H * d, -3.0)
        assert bool((bws[:MARGIN + off] == 0x5A).all()) and bool((bws[MARGIN + off + need:] == 0x5A).all())
    bk, k = _guarded((L, H, T, d), torch.bfloat16, 7.0)
    bv, v = _guarded((L, H, T, d), torch.bfloat16, 7.0)
    kvc.kvc_apply_segmented(src, st, kvc.Segments([0, 100, 333], [5, 0, -40]), rope, kvc.Cache(k, v))
    torch.cuda.synchronize()
    assert _intact(bk, L * H * T * d, 7.0) and _intact(bv, L * H * T * d, 7.0)
