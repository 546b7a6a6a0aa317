"""kvc_chain_fused against kvc_chain: the fused pass must give the hop-by-hop result bit for bit
(every hop rounds to bf16 before it feeds the next), and therefore inherits kvc_chain's parity with
the oracle; the first hop is also compared with the oracle directly."""
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
CFG_P = wl.CONFIGS["vlm_16k"].scaled(name="vlm_small", L=2, H=2, T=2005, image_spans=((512, 1024),))
CFG_R64 = wl.CONFIGS["llama70b_32k"].scaled(name="r64_small", L=1, H=3, T=777, n_agents=8)


@pytest.fixture(autouse=True)
def _clean():
    kvc.kvc_status_reset()
    kvc.kvc_set_path(kvc.KVC_PATH_AUTO)
    yield
    kvc.kvc_set_path(kvc.KVC_PATH_AUTO)
    assert kvc.kvc_status_poll() == 0


def _both(cfg, states_cpu, pl, pairing=kvc.KVC_ROPE_HALF, force_tc=True):
    rope = kvc.Rope(cfg.theta, pairing)
    src_cpu = hp.make_cache(cfg)
    src = hp.to_dev(src_cpu, DEV)
    states = [hp.state_to_dev(s, DEV) for s in states_cpu]
    n = len(pl)
    ref = [hp.empty_dst(src_cpu, cfg, DEV, table_tag=60 + a, fill=2.0) for a in range(1, n)]
    got = [kvc.Cache(torch.full_like(o.k, 2.0), torch.full_like(o.v, 2.0), T=o.T if o.page_table is not None else None,
                     page_table=o.page_table) for o in ref]
    kvc.kvc_chain(src, pl, states, rope, ref)
    ws = torch.empty(max(kvc.kvc_chain_workspace_bytes(src, n), 128), dtype=torch.uint8, device=DEV)
    k0 = src.k.clone()
    if force_tc:
        kvc.kvc_set_path(kvc.KVC_PATH_TC)       # the fused kernel or an error, no silent hop-by-hop
    kvc.kvc_chain_fused(src, pl, states, rope, got, ws)
    torch.cuda.synchronize()
    kvc.kvc_set_path(kvc.KVC_PATH_AUTO)
    assert torch.equal(src.k, k0)                # agent 0 stays exact
    for a, (g, r) in enumerate(zip(got, ref)):
        assert torch.equal(g.k, r.k), f"K of hop {a + 1}"
        assert torch.equal(g.v, r.v), f"V of hop {a + 1}"
    return src_cpu, got


@pytest.mark.parametrize("cfg", [CFG_S, CFG_P, CFG_R64], ids=lambda c: c.name)
def test_fused_chain_equals_hop_by_hop(cfg):
    pl = wl.prefix_lengths(cfg)
    states = [hp.make_state(cfg, hop=a) for a in range(1, cfg.n_agents)]
    src_cpu, got = _both(cfg, states, pl)
    # first hop against the oracle as well
    osrc = hp.oracle_cache(src_cpu)
    odst = osrc.empty_like(page_table=None if got[0].page_table is None else got[0].page_table.cpu().numpy())
    odst, rk, rv = orc.apply(osrc, hp.oracle_state(states[0]), pl[1] - pl[0], hp.inv_freq(cfg), dst=odst, want_ref=True)
    assert hp.tol_ratio(hp.logical_bits(got[0], "k"), rk) <= 1.0 and hp.tol_ratio(hp.logical_bits(got[0], "v"), rv) <= 1.0


def test_fused_chain_partial_coverage_empty_hop_zero_shift_interleaved():
    cfg = CFG_S.scaled(T=700, n_agents=5)
    pl = [100, 100, 260, 131, 131]                       # shifts 0, +160, -129, 0
    states = [hp.make_state(cfg, hop=1, n_cov=300), kvc.State.empty(), hp.make_state(cfg, hop=3, r=16, n_cov=699),
              hp.make_state(cfg, hop=4, basis_dtype=torch.bfloat16)]
    _both(cfg, states, pl)
    _both(cfg, states, pl, pairing=kvc.KVC_ROPE_INTERLEAVED)


def test_fused_chain_falls_back_outside_its_limits():
    cfg = CFG_S.scaled(T=300, n_agents=2)
    pl = [64, 200]
    states = [hp.make_state(cfg, hop=1)]
    _both(cfg, states, pl, force_tc=False)               # one hop: nothing to fuse, runs as kvc_chain
    src = hp.to_dev(hp.make_cache(cfg), DEV)
    out = [hp.empty_dst(hp.make_cache(cfg), cfg, DEV)]
    ws = torch.empty(1 << 20, dtype=torch.uint8, device=DEV)
    kvc.kvc_set_path(kvc.KVC_PATH_TC)
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_chain_fused(src, pl, [hp.state_to_dev(states[0], DEV)], kvc.Rope(cfg.theta), out, ws)
    assert e.value.code == kvc.KVC_E_UNSUPPORTED
    kvc.kvc_set_path(kvc.KVC_PATH_AUTO)
    # a workspace that is too small is an error, not a fallback
    cfg3 = CFG_S.scaled(T=300, n_agents=3)
    st3 = [hp.state_to_dev(hp.make_state(cfg3, hop=a), DEV) for a in (1, 2)]
    outs = [hp.empty_dst(hp.make_cache(cfg3), cfg3, DEV) for _ in range(2)]
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_chain_fused(src, [64, 200, 90], st3, kvc.Rope(cfg.theta), outs, ws[:256])
    assert e.value.code == kvc.KVC_E_WORKSPACE
