"""GPU parity of kvc_apply_multi (Eq. 8 with token-wise weights) against the fp64 oracle.

Element by element on seeded inputs: bf16 results, |gpu - ref| <= 2^-7 |ref| + 1e-3 with ref the
oracle's value before rounding; rows no anchor covers are compared bit for bit.
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

CFG_S = wl.CONFIGS["llama8b_8k"].scaled(name="8b_small", L=2, H=2, T=1000)
CFG_P = wl.CONFIGS["vlm_16k"].scaled(name="vlm_small", L=2, H=2, T=1301, image_spans=())


@pytest.fixture(autouse=True)
def _clean_status():
    kvc.kvc_status_reset()
    yield
    assert kvc.kvc_status_poll() == 0


def _weights(n_anchors, T, seed, tag):
    """Token-wise weights [V, T_pad] fp32: positive, columns sum to one; zero padding."""
    tp = kvc.kvc_multi_tpad(T)
    w = wl.noise((n_anchors, T), seed, 300 + tag, "cpu").abs() + 0.05
    w = w / w.sum(dim=0, keepdim=True)
    out = torch.zeros(n_anchors, tp, dtype=torch.float32)
    out[:, :T] = w
    return out


def _anchors(cfg, ranks, n_covs):
    return [hp.make_state(cfg, hop=v + 1, r=r, n_cov=n) for v, (r, n) in enumerate(zip(ranks, n_covs))]


def _run(cfg, src_cpu, anchors, wk, wv, shift, in_place=False, pairing=kvc.KVC_ROPE_HALF):
    src = hp.to_dev(src_cpu, DEV)
    dst = src if in_place else hp.empty_dst(src_cpu, cfg, DEV, fill=-7.0)
    dev_anchors = [hp.state_to_dev(a, DEV) for a in anchors]
    ws = torch.empty(max(kvc.kvc_multi_workspace_bytes(src, dev_anchors), 128), dtype=torch.uint8, device=DEV)
    mv = lambda t: None if t is None else t.to(DEV)
    kvc.kvc_apply_multi(src, dev_anchors, mv(wk), mv(wv), shift, kvc.Rope(cfg.theta, pairing), dst, ws)
    torch.cuda.synchronize()
    return dst


def _oracle(cfg, src_cpu, anchors, wk, wv, shift, dst_table=None, pairing=orc.ROPE_HALF):
    osrc = hp.oracle_cache(src_cpu)
    odst = osrc.empty_like(page_table=dst_table)
    inv = hp.inv_freq(cfg)
    refs = {"k": [], "v": []}
    for l in range(cfg.L):
        for h in range(cfg.H):
            for which, w in (("k", wk), ("v", wv)):
                ref, out = orc.apply_multi_slab(
                    osrc.get_bits(which, l, h), None if w is None else w.numpy()[:, :cfg.T],
                    [getattr(a, "coeff_" + which)[l, h].numpy() for a in anchors],
                    [getattr(a, "basis_" + which)[l, h].to(torch.float32).numpy() for a in anchors],
                    [a.n_cov for a in anchors], shift, inv, which == "k", pairing)
                odst.put_bits(which, l, h, out)
                refs[which].append(ref)
    shape = (cfg.L, cfg.H, cfg.T, cfg.d)
    return odst, np.stack(refs["k"]).reshape(shape), np.stack(refs["v"]).reshape(shape)


def _check(dst, odst, ref_k, ref_v):
    gk, gv = hp.logical_bits(dst, "k"), hp.logical_bits(dst, "v")
    rk, rv = hp.tol_ratio(gk, ref_k), hp.tol_ratio(gv, ref_v)
    assert rk <= 1.0 and rv <= 1.0, (rk, rv)
    assert hp.ulp_mismatch_fraction(gk, hp.logical_bits(odst, "k")) < 2e-2
    assert hp.ulp_mismatch_fraction(gv, hp.logical_bits(odst, "v")) < 2e-2


@pytest.mark.parametrize("cfg", [CFG_S, CFG_P], ids=lambda c: c.name)
@pytest.mark.parametrize("ranks", [(32, 32, 32), (16, 64, 32, 8), (64, 64, 64, 64, 64)], ids=["3x32", "mixed", "5x64"])
def test_apply_multi_weighted(cfg, ranks):
    T = cfg.T
    anchors = _anchors(cfg, ranks, [T] * len(ranks))
    src_cpu = hp.make_cache(cfg)
    wk, wv = _weights(len(ranks), T, cfg.seed, 0), _weights(len(ranks), T, cfg.seed, 1)
    shift = -137
    dst = _run(cfg, src_cpu, anchors, wk, wv, shift)
    assert kvc.kvc_last_path() == kvc.KVC_PATH_TC
    odst, rk, rv = _oracle(cfg, src_cpu, anchors, wk, wv, shift, dst_table=None if dst.page_table is None else dst.page_table.cpu().numpy())
    _check(dst, odst, rk, rv)


def test_apply_multi_unit_weights_partial_coverage_in_place():
    cfg = CFG_S
    anchors = _anchors(cfg, (32, 32, 16), (cfg.T, 300, 129))
    src_cpu = hp.make_cache(cfg)
    for shift in (0, 64):
        dst = _run(cfg, src_cpu, anchors, None, None, shift, in_place=True)
        odst, rk, rv = _oracle(cfg, src_cpu, anchors, None, None, shift)
        _check(dst, odst, rk, rv)
    # no anchor reaches beyond row 700: rows above keep the source bit for bit at shift 0
    anchors = _anchors(cfg, (32, 32), (700, 650))
    dst = _run(cfg, src_cpu, anchors, None, None, 0)
    sk, sv = hp.logical_bits(src_cpu, "k"), hp.logical_bits(src_cpu, "v")
    gk, gv = hp.logical_bits(dst, "k"), hp.logical_bits(dst, "v")
    assert np.array_equal(gk[:, :, 700:], sk[:, :, 700:]) and np.array_equal(gv[:, :, 700:], sv[:, :, 700:])
    odst, rk, rv = _oracle(cfg, src_cpu, anchors, None, None, 0)
    _check(dst, odst, rk, rv)


def test_apply_multi_one_anchor_is_apply():
    cfg = CFG_P.scaled(T=517)
    anchors = _anchors(cfg, (32,), (cfg.T,))
    src_cpu = hp.make_cache(cfg)
    shift = 33
    dst = _run(cfg, src_cpu, anchors, None, None, shift)
    src = hp.to_dev(src_cpu, DEV)
    one = kvc.Cache(torch.empty_like(dst.k), torch.empty_like(dst.v), T=dst.T, page_table=dst.page_table)
    kvc.kvc_apply(src, hp.state_to_dev(anchors[0], DEV), shift, kvc.Rope(cfg.theta), one)
    torch.cuda.synchronize()
    assert np.array_equal(hp.logical_bits(dst, "k"), hp.logical_bits(one, "k"))
    assert np.array_equal(hp.logical_bits(dst, "v"), hp.logical_bits(one, "v"))


def test_apply_multi_interleaved_pairing_and_bf16_basis():
    cfg = CFG_S.scaled(T=260)
    anchors = [hp.make_state(cfg, hop=v + 1, r=32, basis_dtype=torch.bfloat16) for v in range(2)]
    src_cpu = hp.make_cache(cfg)
    wk, wv = _weights(2, cfg.T, cfg.seed, 2), _weights(2, cfg.T, cfg.seed, 3)
    dst = _run(cfg, src_cpu, anchors, wk, wv, 75, pairing=kvc.KVC_ROPE_INTERLEAVED)
    odst, rk, rv = _oracle(cfg, src_cpu, anchors, wk, wv, 75, pairing=orc.ROPE_INTERLEAVED)
    _check(dst, odst, rk, rv)


def test_apply_multi_limits_and_empty():
    cfg = CFG_S.scaled(T=200)
    src_cpu = hp.make_cache(cfg)
    src = hp.to_dev(src_cpu, DEV)
    dst = hp.empty_dst(src_cpu, cfg, DEV)
    rope = kvc.Rope(cfg.theta)
    ws = torch.empty(1 << 22, dtype=torch.uint8, device=DEV)
    # eleven rank blocks: more than the kernel takes
    many = [hp.state_to_dev(a, DEV) for a in _anchors(cfg, (64, 64, 64, 64, 64, 32), [cfg.T] * 6)]
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_apply_multi(src, many, None, None, 0, rope, dst, ws)
    assert e.value.code == kvc.KVC_E_UNSUPPORTED
    # a workspace that is too small
    two = [hp.state_to_dev(a, DEV) for a in _anchors(cfg, (32, 32), [cfg.T] * 2)]
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_apply_multi(src, two, None, None, 0, rope, dst, ws[:1024])
    assert e.value.code == kvc.KVC_E_WORKSPACE
    # no anchors / only empty anchors: the aligned source, as kvc_apply with an empty state
    for deltas in ([], [kvc.State.empty()]):
        kvc.kvc_apply_multi(src, deltas, None, None, 19, rope, dst, ws)
        torch.cuda.synchronize()
        ref = hp.empty_dst(src_cpu, cfg, DEV)
        kvc.kvc_apply(src, kvc.State.empty(), 19, rope, ref)
        torch.cuda.synchronize()
        assert torch.equal(dst.k, ref.k) and torch.equal(dst.v, ref.v)
