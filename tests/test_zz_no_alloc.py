"""The no-allocation state update (kvc_state_update_noalloc) against kvc_state_update.

Some integrations cannot call cudaMalloc where they need a state update (an engine plugin
living inside a memory pool that was sized at start-up; a process whose GPU memory is all
committed to the KV pool), so the library carries a fixed scratch array for them.  This
file checks, through the C ABI, that the variant produces what the workspace-taking entry
point produces -- twice in a row, with different inputs, because the shared array keeps
the previous call's contents -- and that it refuses problems beyond its capacity.
It is collected last on purpose: a run that stops at the first failure has by then
executed every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import paper_2609_34060_b200 as kvc
from paper_2609_34060_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _edge(cfg, seed):
    """Source and target caches of one edge: generator draws only (the two entry points are
    compared with each other, so any bf16 pair will do; a low-rank-plus-noise pair keeps the
    fitted subspace well defined)."""
    c = cfg.scaled(seed=seed)
    k0, v0 = wl.base_cache(c, "cpu")
    s = wl.hop_state(c, 1, "cpu")
    dk = torch.matmul(s["coeff_k"], s["basis_k"]) + 1e-3 * wl.noise(k0.shape, seed, 1)
    dv = torch.matmul(s["coeff_v"], s["basis_v"]) + 1e-3 * wl.noise(v0.shape, seed, 2)
    src = kvc.Cache(k0.to(DEV), v0.to(DEV))
    tgt = kvc.Cache((k0.float() + dk).to(torch.bfloat16).to(DEV), (v0.float() + dv).to(torch.bfloat16).to(DEV))
    return src, tgt


def _fresh_state(cfg):
    L, H, T, d, r = cfg.L, cfg.H, cfg.T, cfg.d, cfg.r
    return kvc.State(torch.zeros(L, H, T, r, device=DEV), torch.zeros(L, H, T, r, device=DEV),
                     torch.zeros(L, H, r, d, device=DEV), torch.zeros(L, H, r, d, device=DEV))


def _compare(a: "kvc.State", b: "kvc.State"):
    for ca, cb, ba, bb in ((a.coeff_k, b.coeff_k, a.basis_k, b.basis_k), (a.coeff_v, b.coeff_v, a.basis_v, b.basis_v)):
        Ba, Bb = ba.double().cpu().numpy(), bb.double().cpu().numpy()
        Ca, Cb = ca.double().cpu().numpy(), cb.double().cpu().numpy()
        assert np.abs(Ba).max() > 0.05                      # something was written
        # same subspace (projector) and same correction coeff . basis, to the tolerances the
        # fit-mode tests use for a fitted state
        P = np.einsum("lhqc,lhqe->lhce", Ba, Ba) - np.einsum("lhqc,lhqe->lhce", Bb, Bb)
        assert np.sqrt((P ** 2).sum(axis=(2, 3))).max() <= 1e-2
        Ra, Rb = np.einsum("lhtq,lhqc->lhtc", Ca, Ba), np.einsum("lhtq,lhqc->lhtc", Cb, Bb)
        assert np.abs(Ra - Rb).max() <= 1e-3 * max(1.0, np.abs(Rb).max())


def test_noalloc_matches_workspace_variant_twice_in_a_row():
    cfg = wl.CONFIGS["llama8b_8k"].scaled(name="noalloc", L=2, H=3, T=450)
    rope = kvc.Rope(cfg.theta)
    kvc.kvc_status_reset()
    for call, (seed, shift) in enumerate(((21, 37), (22, -120))):
        src, tgt = _edge(cfg, seed)
        want, got = _fresh_state(cfg), _fresh_state(cfg)
        ws = torch.empty(kvc.kvc_workspace_bytes(tgt, want, kvc.KVC_FIT), dtype=torch.uint8, device=DEV)
        kvc.kvc_state_update(src, tgt, shift, rope, want, kvc.KVC_FIT, workspace=ws)
        kvc.kvc_state_update_noalloc(src, tgt, shift, rope, got, kvc.KVC_FIT)
        torch.cuda.synchronize()
        _compare(got, want)
    # PROJECT mode needs no scratch and goes through the same entry point
    src, tgt = _edge(cfg, 23)
    want, got = _fresh_state(cfg), _fresh_state(cfg)
    basis = wl.hop_state(cfg, 2, DEV)
    for s in (want, got):
        s.basis_k.copy_(basis["basis_k"])
        s.basis_v.copy_(basis["basis_v"])
    kvc.kvc_state_update(src, tgt, 5, rope, want, kvc.KVC_PROJECT)
    kvc.kvc_state_update_noalloc(src, tgt, 5, rope, got, kvc.KVC_PROJECT)
    torch.cuda.synchronize()
    assert torch.allclose(got.coeff_k, want.coeff_k, rtol=0, atol=1e-5)
    assert torch.allclose(got.coeff_v, want.coeff_v, rtol=0, atol=1e-5)
    assert kvc.kvc_status_poll() == 0


def test_noalloc_rejects_problems_beyond_its_capacity():
    # L*H = 65 > 64 at d = 128: refused with its own status code, nothing launched
    cfg = wl.CONFIGS["llama8b_8k"].scaled(name="too_big", L=13, H=5, T=16)
    src, tgt = _edge(cfg, 5)
    st = _fresh_state(cfg)
    assert kvc.kvc_workspace_bytes(tgt, st, kvc.KVC_FIT) > kvc.KVC_STATIC_SCRATCH_BYTES
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_state_update_noalloc(src, tgt, 0, kvc.Rope(cfg.theta), st, kvc.KVC_FIT)
    assert e.value.code == -8 and "scratch" in str(e.value)
    torch.cuda.synchronize()
    assert float(st.basis_k.abs().max()) == 0.0
    # the same geometry at the capacity limit (L*H = 64) is accepted
    cfg = cfg.scaled(L=16, H=4)
    src, tgt = _edge(cfg, 6)
    st = _fresh_state(cfg)
    for mode in (kvc.KVC_FIT, kvc.KVC_FIT_FAST):
        st = _fresh_state(cfg)
        assert kvc.KVC_STATIC_SCRATCH_BYTES - 1024 <= kvc.kvc_workspace_bytes(tgt, st, mode) <= kvc.KVC_STATIC_SCRATCH_BYTES
        kvc.kvc_state_update_noalloc(src, tgt, 0, kvc.Rope(cfg.theta), st, mode)
        torch.cuda.synchronize()
        assert float(st.basis_k.abs().max()) > 0.05


def test_noalloc_takes_no_device_memory_after_its_first_call_and_checks_arguments_first():
    cfg = wl.CONFIGS["tiny"]
    src, tgt = _edge(cfg, 31)
    rope = kvc.Rope(cfg.theta)
    st = _fresh_state(cfg)
    kvc.kvc_state_update_noalloc(src, tgt, 0, rope, st, kvc.KVC_FIT)        # first call: the array is resolved
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    for mode in (kvc.KVC_FIT, kvc.KVC_FIT_FAST, kvc.KVC_PROJECT):
        kvc.kvc_state_update_noalloc(src, tgt, 3, rope, st, mode)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    # an invalid call gets its own error even when it is also too large, and writes nothing
    big = wl.CONFIGS["llama8b_8k"].scaled(name="too_big", L=13, H=5, T=16)
    bsrc, btgt = _edge(big, 5)
    bst = _fresh_state(big)
    bst.n_cov = big.T + 1
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_state_update_noalloc(bsrc, btgt, 0, kvc.Rope(big.theta), bst, kvc.KVC_FIT)
    assert e.value.code != -8
