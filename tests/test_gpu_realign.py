"""GPU parity of kvc_state_realign (App. A.2: a stored correction re-aligned when reused) against the
fp64 oracle, and the recurring-prefix use it is for: a correction profiled once at one pair of
positions, stored in canonical coordinates, and reused at another pair of positions."""
import numpy as np
import pytest
import torch

import paper_2609_34060_b200 as kvc
from paper_2609_34060_b200 import workloads as wl
from oracle import kvc_oracle as orc

import helpers as hp

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

CFG_S = wl.CONFIGS["llama8b_8k"].scaled(name="8b_small", L=2, H=2, T=600, r=8)
CFG_T = wl.CONFIGS["tiny"]


@pytest.mark.parametrize("cfg", [CFG_S, CFG_T], ids=lambda c: c.name)
@pytest.mark.parametrize("pairing", [kvc.KVC_ROPE_HALF, kvc.KVC_ROPE_INTERLEAVED], ids=["half", "interleaved"])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_realign_matches_the_oracle(cfg, pairing, dtype):
    st = hp.state_to_dev(hp.make_state(cfg, hop=1, basis_dtype=dtype), DEV)
    inv = hp.inv_freq(cfg)
    for shift in (0, 211, -75):
        out = kvc.kvc_state_realign(st, shift, kvc.Rope(cfg.theta, pairing))
        torch.cuda.synchronize()
        ref = orc.realign_basis(st.basis_k.to(torch.float32).cpu().numpy(), shift, inv,
                                orc.ROPE_HALF if pairing == kvc.KVC_ROPE_HALF else orc.ROPE_INTERLEAVED)
        got = out.basis_k.to(torch.float32).cpu().numpy().astype(np.float64)
        tol = 2e-6 if dtype == torch.float32 else 2.0 ** -8          # float32 rotation / one bf16 rounding
        assert np.max(np.abs(got - ref)) <= tol * max(1.0, np.max(np.abs(ref)))
        if shift == 0:
            assert torch.equal(out.basis_k, st.basis_k)
        assert out.coeff_k.data_ptr() == st.coeff_k.data_ptr() and out.basis_v.data_ptr() == st.basis_v.data_ptr()
    # in place
    keep = st.basis_k.clone()
    kvc.kvc_state_realign(st, 33, kvc.Rope(cfg.theta, pairing), out=st.basis_k)
    kvc.kvc_state_realign(st, -33, kvc.Rope(cfg.theta, pairing), out=st.basis_k)
    torch.cuda.synchronize()
    tol = 1e-5 if dtype == torch.float32 else 2.0 ** -6
    assert torch.max(torch.abs(st.basis_k.float() - keep.float())).item() <= tol


def test_correction_profiled_once_reused_at_other_positions():
    """Profile: fit the key/value deviation of a recurring prefix relation at positions (p_s, p_t) and
    store it canonically (re-aligned by -p_t).  Reuse: another request meets the same relation at
    (p_s', p_t'); the stored correction re-aligned by p_t' and applied to the new source with shift
    p_t' - p_s' must give the oracle's  Rot(src') + Rot_{p_t'}(canonical correction)."""
    cfg = CFG_S
    L, H, T, d, r = cfg.L, cfg.H, cfg.T, cfg.d, cfg.r
    rope = kvc.Rope(cfg.theta)
    inv = hp.inv_freq(cfg)
    p_s, p_t, p_s2, p_t2 = 40, 135, 300, 512
    true = hp.make_state(cfg, hop=3)                    # the relation's deviation, in canonical coordinates
    # profiling request: target = bf16(Rot(src) + Rot_{p_t}(c . B)) by the oracle
    src1_cpu = hp.make_cache(cfg)
    o1 = hp.oracle_cache(src1_cpu)
    prof = orc.State(true.coeff_k.numpy(), true.coeff_v.numpy(),
                     orc.realign_basis(true.basis_k.numpy(), p_t, inv), true.basis_v.numpy())
    tgt1 = orc.apply(o1, prof, p_t - p_s, inv)
    mk = lambda a: torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16)
    src1, tgt1_dev = hp.to_dev(src1_cpu, DEV), kvc.Cache(mk(tgt1.k).to(DEV), mk(tgt1.v).to(DEV))
    st = kvc.State(torch.empty(L, H, T, r, device=DEV), torch.empty(L, H, T, r, device=DEV),
                   torch.empty(L, H, r, d, device=DEV), torch.empty(L, H, r, d, device=DEV))
    ws = torch.empty(kvc.kvc_workspace_bytes(tgt1_dev, st, kvc.KVC_FIT), dtype=torch.uint8, device=DEV)
    kvc.kvc_state_update(src1, tgt1_dev, p_t - p_s, rope, st, kvc.KVC_FIT, workspace=ws)
    stored = kvc.kvc_state_realign(st, -p_t, rope)      # canonical storage
    # reuse on another request (another seed), at other positions
    cfg2 = cfg.scaled(seed=cfg.seed + 5)
    src2_cpu = hp.make_cache(cfg2)
    src2 = hp.to_dev(src2_cpu, DEV)
    reuse = kvc.kvc_state_realign(stored, p_t2, rope)
    dst = hp.empty_dst(src2_cpu, cfg2, DEV)
    kvc.kvc_apply(src2, reuse, p_t2 - p_s2, rope, dst)
    torch.cuda.synchronize()
    assert kvc.kvc_status_poll() == 0
    # oracle: the same three steps - fit on the same profiling pair, store canonically, re-align to p_t'
    ofit, _ = orc.state_update(o1, tgt1, p_t - p_s, inv, r=r, mode=orc.FIT)
    canon = orc.realign_basis(ofit.basis_k, -p_t, inv)
    want = orc.State(ofit.coeff_k, ofit.coeff_v, orc.realign_basis(canon, p_t2, inv), ofit.basis_v)
    o2 = hp.oracle_cache(src2_cpu)
    odst, rk, rv = orc.apply(o2, want, p_t2 - p_s2, inv, want_ref=True)
    gk, gv = hp.logical_bits(dst, "k"), hp.logical_bits(dst, "v")
    # (bases may differ in sign between the two eigensolvers; the correction c . B does not)
    assert hp.tol_ratio(gk, rk) <= 1.0
    assert hp.tol_ratio(gv, rv) <= 1.0
