"""GPU parity of the reliability gate (App. A.3, Eqs. 9-11) against the fp64 oracle.

kvc_gate_distance: the squared distance of every anchor, compared with the oracle's Eq. 9 on the same
seeded inputs (the source cache's values are derived by the oracle's arithmetic from generator draws:
values close to anchor 0's reconstruction, far from the others).  kvc_gate_weights: fed seeded numbers
from the host and compared with the oracle's Eqs. 10-11 on the same numbers.
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
CFG_8B_S = wl.CONFIGS["llama8b_8k"].scaled(name="8b_small", L=2, H=2, T=1000)
CFG_VLM_S = wl.CONFIGS["vlm_16k"].scaled(name="vlm_small", L=2, H=2, T=2005, image_spans=())
CFG_R64_S = wl.CONFIGS["llama70b_32k"].scaled(name="r64_small", L=1, H=3, T=777)

PATHS = [kvc.KVC_PATH_GENERIC, kvc.KVC_PATH_AUTO]
PATH_IDS = ["generic", "auto"]


@pytest.fixture(autouse=True)
def _reset_path():
    kvc.kvc_status_reset()
    yield
    kvc.kvc_set_path(kvc.KVC_PATH_AUTO)
    assert kvc.kvc_status_poll() == 0


def _scenario(cfg, n_anchors, noise=0.05):
    """Anchors = independent draws of value factors; the source cache's values are anchor 0's
    reconstruction plus noise, rounded to bf16 (oracle arithmetic on generator draws)."""
    anchors = [hp.make_state(cfg, hop=v + 1) for v in range(n_anchors)]
    src = hp.make_cache(cfg)
    osrc = hp.oracle_cache(src)
    eps = wl.noise((cfg.L, cfg.H, cfg.T, cfg.d), cfg.seed, 77, "cpu").numpy().astype(np.float64)
    c0 = anchors[0].coeff_v.numpy().astype(np.float64)
    b0 = anchors[0].basis_v.numpy().astype(np.float64)
    for l in range(cfg.L):
        for h in range(cfg.H):
            osrc.put_bits("v", l, h, orc.f64_to_bf16_bits(c0[l, h] @ b0[l, h] + noise * eps[l, h]))
    # the device cache is rebuilt from the oracle-side bit patterns (same layout, same table)
    v_new = torch.from_numpy(osrc.v.view(np.int16).copy()).view(torch.bfloat16)
    if src.page_table is None:
        src = kvc.Cache(src.k, v_new)
    else:
        src = kvc.Cache(src.k, v_new, T=src.T, page_table=src.page_table)
    return src, osrc, anchors


def _oracle_dist(cfg, osrc, anchors, k):
    out = []
    for a in anchors:
        c = a.coeff_v.numpy().astype(np.float64)
        b = a.basis_v.to(torch.float32).numpy().astype(np.float64)
        v_src = [np.concatenate([orc.bf16_to_f64(osrc.get_bits("v", l, h)) for h in range(cfg.H)], axis=1)
                 for l in range(cfg.L)]
        v_anc = [np.concatenate([c[l, h] @ b[l, h] for h in range(cfg.H)], axis=1) for l in range(cfg.L)]
        out.append(orc.gate_distance(v_src, v_anc, k))
    return np.array(out)


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
@pytest.mark.parametrize("cfg", [CFG_TINY, CFG_8B_S, CFG_VLM_S, CFG_R64_S], ids=lambda c: c.name)
def test_gate_distance_matches_eq9(cfg, path):
    src_cpu, osrc, anchors = _scenario(cfg, 3)
    kvc.kvc_set_path(path)
    src = hp.to_dev(src_cpu, DEV)
    dev_anchors = [hp.state_to_dev(a, DEV) for a in anchors]
    for k in sorted({cfg.T, cfg.T - 1, max(1, cfg.T // 3), 1}):
        d2 = torch.full((3,), -1.0, dtype=torch.float64, device=DEV)
        kvc.kvc_gate_distance(src, dev_anchors, k, d2)
        torch.cuda.synchronize()
        if path == kvc.KVC_PATH_AUTO and cfg.d == 128:
            assert kvc.kvc_last_path() == kvc.KVC_PATH_TC
        got = np.sqrt(d2.cpu().numpy())
        ref = _oracle_dist(cfg, osrc, anchors, k)
        # split-bf16 products (2^-16 relative per product, random sign) under a float32 sum: the
        # distance moves by far less than 1e-4 relative; 1e-3 would already mean a dropped term
        assert np.all(np.abs(got - ref) <= 1e-4 * ref + 1e-6), (k, got, ref)
        assert ref[0] < 0.2 * ref[1:].min()            # the scenario has one clearly matching anchor


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_gate_distance_edges(path):
    cfg = CFG_8B_S.scaled(T=300)
    src_cpu, osrc, anchors = _scenario(cfg, 2)
    kvc.kvc_set_path(path)
    src = hp.to_dev(src_cpu, DEV)
    dev_anchors = [hp.state_to_dev(a, DEV) for a in anchors]
    d2 = torch.full((2,), -1.0, dtype=torch.float64, device=DEV)
    kvc.kvc_gate_distance(src, dev_anchors, 0, d2)             # empty prefix: zero distance
    torch.cuda.synchronize()
    assert d2.cpu().tolist() == [0.0, 0.0]
    # an anchor whose stored length is below the comparison length is not compatible
    short = kvc.State(dev_anchors[1].coeff_k[:, :, :200].contiguous(), dev_anchors[1].coeff_v[:, :, :200].contiguous(),
                      dev_anchors[1].basis_k, dev_anchors[1].basis_v)
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_gate_distance(src, [dev_anchors[0], short], 250, d2)
    assert e.value.code == kvc.KVC_E_SHAPE
    kvc.kvc_gate_distance(src, [dev_anchors[0], short], 200, d2)   # ... and is at or below its length
    torch.cuda.synchronize()
    ref = _oracle_dist(cfg, osrc, anchors, 200)
    assert np.all(np.abs(np.sqrt(d2.cpu().numpy()) - ref) <= 1e-4 * ref + 1e-6)
    # an anchor with bf16 basis and no key factors at all
    a = dev_anchors[1]
    vonly = kvc.State.values_only(a.coeff_v, a.basis_v.to(torch.bfloat16))
    d1 = torch.zeros(1, dtype=torch.float64, device=DEV)
    kvc.kvc_gate_distance(src, [vonly], cfg.T, d1)
    torch.cuda.synchronize()
    b16 = kvc.State(anchors[1].coeff_k, anchors[1].coeff_v, anchors[1].basis_k,
                    anchors[1].basis_v.to(torch.bfloat16).to(torch.float32))
    ref = _oracle_dist(cfg, osrc, [b16], cfg.T)
    assert abs(np.sqrt(d1.item()) - ref[0]) <= 1e-4 * ref[0]


def test_gate_weights_match_eq10_eq11():
    rng = np.random.default_rng(5)
    cases = [rng.uniform(0.0, 30.0, size=n) ** 2 for n in (2, 3, 5, 8, 33, 100)]
    cases.append(np.full(4, 7.0))                       # equal distances: uniform weights, entropy 1
    cases.append(np.array([0.0, 1e6, 1e6]))             # one distinctive match: one-hot, entropy 0
    cases.append(np.array([1e8, 1e8 + 1e-3]))           # large distances: the softmax must not underflow to 0/0
    for d2 in cases:
        n = d2.size
        dev = torch.from_numpy(d2).to(DEV)
        g = torch.empty(n, dtype=torch.float64, device=DEV)
        ent = torch.empty(1, dtype=torch.float64, device=DEV)
        for temp in (1.0, 2.5):
            kvc.kvc_gate_weights(dev, g, ent, temperature=temp)
            torch.cuda.synchronize()
            ref_g = orc.gate_weights(np.sqrt(d2), temp)
            ref_h = orc.normalized_entropy(ref_g)
            assert np.allclose(g.cpu().numpy(), ref_g, rtol=1e-12, atol=1e-15)
            assert abs(ent.item() - ref_h) <= 1e-12
    g = torch.empty(1, dtype=torch.float64, device=DEV)
    with pytest.raises(kvc.KvcError):                   # fewer than two compatible anchors: dense prefill
        kvc.kvc_gate_weights(torch.zeros(1, dtype=torch.float64, device=DEV), g, g)


def test_gate_end_to_end_accepts_the_matching_anchor():
    cfg = CFG_8B_S.scaled(T=640)
    src_cpu, osrc, anchors = _scenario(cfg, 4, noise=0.02)
    src = hp.to_dev(src_cpu, DEV)
    d2 = torch.empty(4, dtype=torch.float64, device=DEV)
    g = torch.empty(4, dtype=torch.float64, device=DEV)
    ent = torch.empty(1, dtype=torch.float64, device=DEV)
    kvc.kvc_gate_distance(src, [hp.state_to_dev(a, DEV) for a in anchors], cfg.T, d2)
    kvc.kvc_gate_weights(d2, g, ent)
    torch.cuda.synchronize()
    ref_d = _oracle_dist(cfg, osrc, anchors, cfg.T)
    ref_g = orc.gate_weights(ref_d)
    # distances differ by tens of units here, so the weights are one-hot on both sides
    assert int(torch.argmax(g).item()) == int(np.argmax(ref_g)) == 0
    assert g[0].item() > 1.0 - 1e-9 and ent.item() < 1e-6 and orc.normalized_entropy(ref_g) < 1e-6


def test_base_factorisation_then_gate_is_the_truncation_residual():
    """An anchor's base cache factorised by itself (src = NULL, FIT) and compared with itself: the
    squared gate distance is what a rank-r truncation leaves, sum over value slabs of the
    eigenvalues of V^T V beyond the r-th (Eckart-Young), computed here by a library eigensolver."""
    cfg = CFG_8B_S.scaled(L=1, H=2, T=400)
    r = 32
    cache_cpu = hp.make_cache(cfg)
    cache = hp.to_dev(cache_cpu, DEV)
    L, H, T, d = cfg.L, cfg.H, cfg.T, cfg.d
    st = kvc.State(torch.empty(L, H, T, r, device=DEV), torch.empty(L, H, T, r, device=DEV),
                   torch.empty(L, H, r, d, device=DEV), torch.empty(L, H, r, d, device=DEV))
    ws = torch.empty(kvc.kvc_workspace_bytes(cache, st, kvc.KVC_FIT), dtype=torch.uint8, device=DEV)
    kvc.kvc_state_update(None, cache, 0, kvc.Rope(cfg.theta), st, kvc.KVC_FIT, workspace=ws)
    d2 = torch.empty(1, dtype=torch.float64, device=DEV)
    kvc.kvc_gate_distance(cache, [st], T, d2)
    torch.cuda.synchronize()
    oc = hp.oracle_cache(cache_cpu)
    expect = 0.0
    for l in range(L):
        for h in range(H):
            v = orc.bf16_to_f64(oc.get_bits("v", l, h))
            lam = np.linalg.eigvalsh(v.T @ v)[::-1]
            expect += float(np.sum(lam[r:]))
    assert abs(d2.item() - expect) <= 2e-3 * expect, (d2.item(), expect)
