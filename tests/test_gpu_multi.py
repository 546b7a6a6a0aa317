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


def _oracle_token_weights(cfg, osrc, src_pos, anchors, anchor_pos, temperature=1.0):
    """App. A.3 with the oracle: features of a token = all (layer, head) slabs side by side; keys in
    canonical coordinates on both sides."""
    inv = hp.inv_freq(cfg)
    slabs = [(l, h) for l in range(cfg.L) for h in range(cfg.H)]
    out = {}
    for which in ("k", "v"):
        if which == "k":
            src_feat = orc.canonical_key_features([osrc.get_bits("k", l, h) for l, h in slabs], src_pos, inv)
        else:
            src_feat = np.concatenate([orc.bf16_to_f64(osrc.get_bits("v", l, h)) for l, h in slabs], axis=1)
        w = np.zeros((len(anchors), cfg.T))
        # the softmax runs over the anchors that cover a token: group tokens by the set of covering anchors
        covs = sorted({a.n_cov for a in anchors} | {0, cfg.T})
        for lo, hi in zip(covs[:-1], covs[1:]):
            idx = [v for v, a in enumerate(anchors) if a.n_cov >= hi]
            if not idx or hi <= lo:
                continue
            feats = []
            for v in idx:
                a = anchors[v]
                c = getattr(a, "coeff_" + which).numpy().astype(np.float64)
                b = getattr(a, "basis_" + which).to(torch.float32).numpy().astype(np.float64)
                rec = [c[l, h, lo:hi] @ b[l, h] for l, h in slabs]
                if which == "k":
                    rec = [orc.rope_shift(x, -anchor_pos[v], inv) for x in rec]
                feats.append(np.concatenate(rec, axis=1))
            w[idx, lo:hi] = orc.token_weights(src_feat[lo:hi], feats, temperature)
        out[which] = w
    return out["k"], out["v"]


@pytest.mark.parametrize("cfg", [CFG_S, CFG_P], ids=lambda c: c.name)
def test_token_weights_match_the_oracle(cfg):
    T = cfg.T
    ranks, covs = (32, 32, 64), (T, T, T - 300)
    anchors = _anchors(cfg, ranks, covs)
    anchor_pos = [100, 37, 412]
    src_pos = 250
    # the source cache sits close to anchor 0's base on the first half of the tokens and close to
    # anchor 1's on the second half (oracle arithmetic on generator draws), keys moved to the
    # source's positions
    src_cpu = hp.make_cache(cfg)
    osrc = hp.oracle_cache(src_cpu)
    inv = hp.inv_freq(cfg)
    eps = wl.noise((2, cfg.L, cfg.H, T, cfg.d), cfg.seed, 91, "cpu").numpy().astype(np.float64)
    half = T // 2
    for l in range(cfg.L):
        for h in range(cfg.H):
            for wi, which in enumerate(("k", "v")):
                rec = []
                for v in (0, 1):
                    c = getattr(anchors[v], "coeff_" + which)[l, h].numpy().astype(np.float64)
                    b = getattr(anchors[v], "basis_" + which)[l, h].numpy().astype(np.float64)
                    x = c @ b
                    if which == "k":
                        x = orc.rope_shift(x, src_pos - anchor_pos[v], inv)
                    rec.append(x)
                mix = np.where(np.arange(T)[:, None] < half, rec[0], rec[1]) + 0.3 * eps[wi, l, h]
                osrc.put_bits(which, l, h, orc.f64_to_bf16_bits(mix))
    mk = lambda a: torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16)
    src_cpu = kvc.Cache(mk(osrc.k), mk(osrc.v)) if src_cpu.page_table is None else \
        kvc.Cache(mk(osrc.k), mk(osrc.v), T=T, page_table=src_cpu.page_table)
    src = hp.to_dev(src_cpu, DEV)
    dev_anchors = [hp.state_to_dev(a, DEV) for a in anchors]
    tp = kvc.kvc_multi_tpad(T)
    wk = torch.full((3, tp), -1.0, device=DEV)
    wv = torch.full((3, tp), -1.0, device=DEV)
    ws = torch.empty(kvc.kvc_token_weights_workspace_bytes(src, 3), dtype=torch.uint8, device=DEV)
    for temp in (1.0, 0.25):
        kvc.kvc_token_weights(src, src_pos, dev_anchors, anchor_pos, kvc.Rope(cfg.theta), wk, wv, ws, temperature=temp)
        torch.cuda.synchronize()
        rk, rv = _oracle_token_weights(cfg, osrc, src_pos, anchors, anchor_pos, temp)
        gk, gv = wk.cpu().numpy().astype(np.float64), wv.cpu().numpy().astype(np.float64)
        # scores are float32 means of ~L*H*d terms with split-precision products: 1e-5 absolute on a weight
        assert np.max(np.abs(gk[:, :T] - rk)) <= 2e-5 and np.max(np.abs(gv[:, :T] - rv)) <= 2e-5
        assert np.all(gk[:, T:] == 0) and np.all(gv[:, T:] == 0)               # the padding
        assert np.all(gk[2, T - 300:T] == 0) and np.all(gv[2, T - 300:T] == 0)   # beyond anchor 2's coverage
        assert np.allclose(gk[:, :T].sum(axis=0), 1.0, atol=1e-5)
    # the scenario is token-wise: the first half prefers anchor 0, the second half anchor 1
    assert rk[0, :half].mean() > 0.5 > rk[0, half:].mean() and rv[1, half:].mean() > 0.5 > rv[1, :half].mean()


def test_multi_anchor_pipeline_gate_weights_apply():
    """Gate, token weights and weighted apply chained on the device against the same chain in the oracle."""
    cfg = CFG_S.scaled(T=640)
    T = cfg.T
    base = _anchors(cfg, (32, 32), (T, T))                       # the anchors' base factorisations
    delta = [hp.make_state(cfg, hop=v + 5, r=32) for v in range(2)]   # their stored corrections
    src_cpu = hp.make_cache(cfg)
    osrc = hp.oracle_cache(src_cpu)
    src = hp.to_dev(src_cpu, DEV)
    dev_base = [hp.state_to_dev(a, DEV) for a in base]
    dev_delta = [hp.state_to_dev(a, DEV) for a in delta]
    rope = kvc.Rope(cfg.theta)
    d2 = torch.empty(2, dtype=torch.float64, device=DEV)
    g = torch.empty(2, dtype=torch.float64, device=DEV)
    ent = torch.empty(1, dtype=torch.float64, device=DEV)
    kvc.kvc_gate_distance(src, dev_base, T, d2)
    kvc.kvc_gate_weights(d2, g, ent)
    tp = kvc.kvc_multi_tpad(T)
    wk, wv = torch.empty(2, tp, device=DEV), torch.empty(2, tp, device=DEV)
    ws = torch.empty(kvc.kvc_token_weights_workspace_bytes(src, 2), dtype=torch.uint8, device=DEV)
    kvc.kvc_token_weights(src, 0, dev_base, [0, 0], rope, wk, wv, ws)
    dst = hp.empty_dst(src_cpu, cfg, DEV)
    ws2 = torch.empty(kvc.kvc_multi_workspace_bytes(src, dev_delta), dtype=torch.uint8, device=DEV)
    kvc.kvc_apply_multi(src, dev_delta, wk, wv, 48, rope, dst, ws2)
    torch.cuda.synchronize()
    assert 0.0 <= ent.item() <= 1.0 + 1e-12
    ok_, ov_ = _oracle_token_weights(cfg, osrc, 0, base, [0, 0])
    pad = lambda w: torch.from_numpy(np.pad(w, ((0, 0), (0, tp - T))).astype(np.float32))
    odst, rk, rv = _oracle(cfg, src_cpu, delta, pad(ok_), pad(ov_), 48)
    _check(dst, odst, rk, rv)
