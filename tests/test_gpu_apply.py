"""GPU parity of kvc_apply / kvc_chain / kvc_apply_batch against the fp64 oracle.

Every comparison is element by element on the same seeded inputs.  Results are bf16, so the
bar is |gpu - ref| <= 2^-7 |ref| + 1e-3 with ref the oracle's value before its own rounding;
indexing (paging, untouched rows, empty states) is compared bit for bit.
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
CFG_VLM_S = wl.CONFIGS["vlm_16k"].scaled(name="vlm_small", L=2, H=2, T=2005, image_spans=((512, 1024),))
CFG_R64_S = wl.CONFIGS["llama70b_32k"].scaled(name="r64_small", L=1, H=3, T=777)
CFG_D64_R16 = CFG_TINY.scaled(name="d64_r16", T=300, r=16, prefix=(100, 37))

PATHS = [kvc.KVC_PATH_GENERIC, kvc.KVC_PATH_AUTO]
PATH_IDS = ["generic", "auto"]


@pytest.fixture(autouse=True)
def _reset_path():
    kvc.kvc_status_reset()
    yield
    kvc.kvc_set_path(kvc.KVC_PATH_AUTO)
    assert kvc.kvc_status_poll() == 0


def _run_hop(cfg, src_cpu, st_cpu, shift, path, dst_fill=None, in_place=False, pairing=kvc.KVC_ROPE_HALF):
    kvc.kvc_set_path(path)
    rope = kvc.Rope(cfg.theta, pairing)
    src = hp.to_dev(src_cpu, DEV)
    dst = src if in_place else hp.empty_dst(src_cpu, cfg, DEV, fill=dst_fill)
    st = hp.state_to_dev(st_cpu, DEV)
    kvc.kvc_apply(src, st, shift, rope, dst)
    torch.cuda.synchronize()
    if path == kvc.KVC_PATH_AUTO and cfg.d == 128 and 0 < st.r <= 64 and st.n_cov > 0 and cfg.T > 0:
        assert kvc.kvc_last_path() == kvc.KVC_PATH_TC, "the TMA + tcgen05 kernels should have served this call"
    return src, dst


def _oracle_hop(cfg, src_cpu, st_cpu, shift, dst_table=None, pairing=orc.ROPE_HALF):
    osrc = hp.oracle_cache(src_cpu)
    odst = osrc.empty_like(page_table=dst_table)
    return orc.apply(osrc, hp.oracle_state(st_cpu), shift, hp.inv_freq(cfg), dst=odst, pairing=pairing, want_ref=True)


def _assert_parity(dst, ref_k, ref_v, odst):
    gk, gv = hp.logical_bits(dst, "k"), hp.logical_bits(dst, "v")
    rk, rv = hp.tol_ratio(gk, ref_k), hp.tol_ratio(gv, ref_v)
    assert rk <= 1.0 and rv <= 1.0, (rk, rv)
    # sanity beside the tolerance: almost every element is the oracle's own rounding (the
    # split-precision tensor-core contraction differs from float64 by ~1e-5, which flips a
    # bf16 rounding in a few elements per thousand at rank 64)
    assert hp.ulp_mismatch_fraction(gk, hp.logical_bits(odst, "k")) < 1e-2
    assert hp.ulp_mismatch_fraction(gv, hp.logical_bits(odst, "v")) < 1e-2


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
@pytest.mark.parametrize("cfg", [CFG_TINY, CFG_8B_S, CFG_VLM_S, CFG_R64_S, CFG_D64_R16], ids=lambda c: c.name)
def test_apply_one_hop(cfg, path):
    src_cpu = hp.make_cache(cfg)
    st_cpu = hp.make_state(cfg, 1)
    pl = wl.prefix_lengths(cfg)
    shift = pl[1] - pl[0]
    src, dst = _run_hop(cfg, src_cpu, st_cpu, shift, path, dst_fill=-7.0)
    odst, ref_k, ref_v = _oracle_hop(cfg, src_cpu, st_cpu, shift,
                                     None if dst.page_table is None else dst.page_table.cpu().numpy())
    _assert_parity(dst, ref_k, ref_v, odst)
    # the source is only read
    assert torch.equal(src.k.cpu(), src_cpu.k) and torch.equal(src.v.cpu(), src_cpu.v)
    if dst.page_table is not None:
        # physical pages the destination table does not name, and rows of the last partial
        # page beyond T, keep their fill
        fill = torch.tensor(-7.0, dtype=torch.bfloat16)
        mapped = set(int(p) for p in dst.page_table.cpu())
        for p in range(dst.P):
            if p not in mapped:
                assert torch.all(dst.k[:, p].cpu() == fill) and torch.all(dst.v[:, p].cpu() == fill)
        tail = cfg.T % cfg.page
        if tail:
            last = int(dst.page_table[-1])
            assert torch.all(dst.k[:, last, :, tail:].cpu() == fill)


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
@pytest.mark.parametrize("shift", [0, -211, 512])
@pytest.mark.parametrize("n_cov", [0, 1, 300, 999, 1000])
def test_partial_coverage_and_shifts(path, shift, n_cov):
    cfg = CFG_8B_S
    src_cpu = hp.make_cache(cfg)
    st_cpu = hp.make_state(cfg, 2, n_cov=n_cov) if n_cov else kvc.State.empty()
    if n_cov == 0:   # rank > 0, nothing covered
        full = hp.make_state(cfg, 2)
        st_cpu = kvc.State(None, None, full.basis_k, full.basis_v, n_cov=0)
    src, dst = _run_hop(cfg, src_cpu, st_cpu, shift, path)
    odst, ref_k, ref_v = _oracle_hop(cfg, src_cpu, st_cpu, shift)
    _assert_parity(dst, ref_k, ref_v, odst)
    # rows beyond the covered prefix: values bit-identical; keys bit-identical at shift 0
    assert torch.equal(dst.v[:, :, n_cov:].cpu(), src_cpu.v[:, :, n_cov:])
    if shift == 0:
        assert torch.equal(dst.k[:, :, n_cov:].cpu(), src_cpu.k[:, :, n_cov:])
    elif n_cov < cfg.T:
        assert not torch.equal(dst.k[:, :, n_cov:].cpu(), src_cpu.k[:, :, n_cov:])


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_empty_state_is_bit_identity_with_exotic_patterns(path):
    cfg = CFG_8B_S.scaled(T=130)
    src_cpu = hp.make_cache(cfg)
    pat = torch.tensor([0x8000, 0x7F80, 0xFF80, 0x7FC1, 0x0001, 0x8001, 0x7F7F, 0x0080], dtype=torch.int32)
    src_cpu.k.view(torch.int16)[0, 0, 5, :8] = pat.to(torch.int16)
    src_cpu.v.view(torch.int16)[1, 1, 129, 8:16] = pat.to(torch.int16)
    src, dst = _run_hop(cfg, src_cpu, kvc.State.empty(), 0, path)
    assert np.array_equal(hp.bits_of(dst.k), hp.bits_of(src_cpu.k))
    assert np.array_equal(hp.bits_of(dst.v), hp.bits_of(src_cpu.v))
    # a covered prefix in front of them does not disturb the uncovered rows either
    st = hp.make_state(cfg, 1, n_cov=3)
    src, dst = _run_hop(cfg, src_cpu, st, 0, path)
    assert np.array_equal(hp.bits_of(dst.k)[:, :, 3:], hp.bits_of(src_cpu.k)[:, :, 3:])
    assert np.array_equal(hp.bits_of(dst.v)[:, :, 3:], hp.bits_of(src_cpu.v)[:, :, 3:])


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
@pytest.mark.parametrize("T", [1, 15, 16, 17, 127, 128, 129, 257])
def test_ragged_lengths_paged(path, T):
    cfg = CFG_VLM_S.scaled(T=T, image_spans=())
    src_cpu = hp.make_cache(cfg)
    st_cpu = hp.make_state(cfg, 1)
    src, dst = _run_hop(cfg, src_cpu, st_cpu, 33, path, dst_fill=5.0)
    odst, ref_k, ref_v = _oracle_hop(cfg, src_cpu, st_cpu, 33, dst.page_table.cpu().numpy())
    _assert_parity(dst, ref_k, ref_v, odst)


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_paged_indexing_bit_exact(path):
    # a 16-bit code that is injective in (t, c) inside every (layer, head) slab (T d = 37,504 distinct patterns)
    # and shifted by a slab-dependent constant (16 bits cannot tell all 225,024 elements apart); rank 0,
    # shift 0, two different shuffled tables: the bits must arrive where the destination table says
    L, H, T, d, page, P = 2, 3, 293, 128, 16, 25
    npg = (T + page - 1) // page
    in_slab = torch.arange(T * d, dtype=torch.int64).reshape(1, 1, T, d)
    slab_off = (torch.arange(L * H, dtype=torch.int64) * 7919).reshape(L, H, 1, 1)
    code = ((in_slab + slab_off) % 65536).to(torch.int32)
    code = torch.where(code >= 32768, code - 65536, code).to(torch.int16).expand(L, H, T, d).contiguous()
    assert all(code[l, h].unique().numel() == T * d for l in range(L) for h in range(H))
    pt_s = wl.page_table(npg, P, 3, 0)
    pt_d = wl.page_table(npg, P, 3, 1)
    pool_k = torch.full((L, P, H, page, d), 0x5EAD, dtype=torch.int16)
    pool_v = torch.full((L, P, H, page, d), 0x5EAD, dtype=torch.int16)
    for t in range(T):
        pool_k[:, int(pt_s[t // page]), :, t % page] = code[:, :, t]
        pool_v[:, int(pt_s[t // page]), :, t % page] = code[:, :, t] ^ 0x4000
    src_cpu = kvc.Cache(pool_k.view(torch.bfloat16), pool_v.view(torch.bfloat16), T=T, page_table=pt_s)
    kvc.kvc_set_path(path)
    src = hp.to_dev(src_cpu, DEV)
    dst = kvc.Cache(torch.full_like(src.k, 3.0), torch.full_like(src.v, 3.0), T=T, page_table=pt_d.to(DEV))
    kvc.kvc_apply(src, kvc.State.empty(), 0, kvc.Rope(500000.0), dst)
    torch.cuda.synchronize()
    dk, dv = dst.k.cpu().view(torch.int16), dst.v.cpu().view(torch.int16)
    for t in range(T):
        assert torch.equal(dk[:, int(pt_d[t // page]), :, t % page], code[:, :, t])
        assert torch.equal(dv[:, int(pt_d[t // page]), :, t % page], code[:, :, t] ^ 0x4000)


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_in_place_and_mixed_layouts(path):
    cfg = CFG_8B_S
    src_cpu = hp.make_cache(cfg)
    st_cpu = hp.make_state(cfg, 1)
    _, ref = _run_hop(cfg, src_cpu, st_cpu, 77, path)
    _, inpl = _run_hop(cfg, src_cpu, st_cpu, 77, path, in_place=True)
    assert torch.equal(ref.k, inpl.k) and torch.equal(ref.v, inpl.v)
    # contiguous source -> paged destination gives the same logical cache
    kvc.kvc_set_path(path)
    npg = wl.n_pages(cfg.T, 16)
    pt = wl.page_table(npg, npg + 2, 9, 0).to(DEV)
    dst = kvc.Cache(torch.zeros(cfg.L, npg + 2, cfg.H, 16, cfg.d, dtype=torch.bfloat16, device=DEV),
                    torch.zeros(cfg.L, npg + 2, cfg.H, 16, cfg.d, dtype=torch.bfloat16, device=DEV), T=cfg.T, page_table=pt)
    kvc.kvc_apply(hp.to_dev(src_cpu, DEV), hp.state_to_dev(st_cpu, DEV), 77, kvc.Rope(cfg.theta), dst)
    torch.cuda.synchronize()
    assert np.array_equal(hp.logical_bits(dst, "k"), hp.bits_of(ref.k))
    assert np.array_equal(hp.logical_bits(dst, "v"), hp.bits_of(ref.v))


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_interleaved_pairing_and_bf16_basis(path):
    cfg = CFG_8B_S.scaled(T=200)
    src_cpu = hp.make_cache(cfg)
    st_cpu = hp.make_state(cfg, 1, basis_dtype=torch.bfloat16)
    src, dst = _run_hop(cfg, src_cpu, st_cpu, -45, path, pairing=kvc.KVC_ROPE_INTERLEAVED)
    odst, ref_k, ref_v = _oracle_hop(cfg, src_cpu, st_cpu, -45, pairing=orc.ROPE_INTERLEAVED)
    _assert_parity(dst, ref_k, ref_v, odst)


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_bad_page_id_is_flagged_not_followed(path):
    cfg = CFG_VLM_S.scaled(T=64, image_spans=())
    src_cpu = hp.make_cache(cfg)
    bad = src_cpu.page_table.clone()
    bad[1] = src_cpu.P + 5                         # outside the pool: built on the host
    src_bad = kvc.Cache(src_cpu.k, src_cpu.v, T=cfg.T, page_table=bad)
    kvc.kvc_set_path(path)
    src = hp.to_dev(src_bad, DEV)
    dst = hp.empty_dst(src_cpu, cfg, DEV, fill=9.0)
    kvc.kvc_apply(src, hp.state_to_dev(hp.make_state(cfg, 1), DEV), 5, kvc.Rope(cfg.theta), dst)
    torch.cuda.synchronize()
    assert kvc.kvc_status_poll() & kvc.KVC_FLAG_BAD_PAGE
    kvc.kvc_status_reset()
    # tokens of the bad page were skipped: the destination rows keep their fill
    p = int(dst.page_table[1])
    assert torch.all(dst.k[:, p].cpu() == torch.tensor(9.0, dtype=torch.bfloat16))


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
@pytest.mark.parametrize("cfg", [CFG_TINY, CFG_8B_S, CFG_VLM_S], ids=lambda c: c.name)
def test_chain(cfg, path):
    pl = wl.prefix_lengths(cfg)
    n = cfg.n_agents
    a0_cpu = hp.make_cache(cfg)
    states_cpu = [hp.make_state(cfg, a) for a in range(1, n)]
    tables = None
    if cfg.paged:
        tables = [wl.page_table(a0_cpu.page_table.numel(), a0_cpu.P, cfg.seed, 60 + a) for a in range(1, n)]
    # oracle: the chained recursion, bf16 at every hop
    o0 = hp.oracle_cache(a0_cpu)
    oouts, orefs = orc.chain(o0, pl, [hp.oracle_state(s) for s in states_cpu], hp.inv_freq(cfg),
                             dst_tables=None if tables is None else [t.numpy() for t in tables], want_ref=True)
    kvc.kvc_set_path(path)
    rope = kvc.Rope(cfg.theta)
    a0 = hp.to_dev(a0_cpu, DEV)
    states = [hp.state_to_dev(s, DEV) for s in states_cpu]

    def fresh_outs():
        if not cfg.paged:
            return [kvc.Cache(torch.zeros_like(a0.k), torch.zeros_like(a0.v)) for _ in range(n - 1)]
        return [kvc.Cache(torch.zeros_like(a0.k), torch.zeros_like(a0.v), T=cfg.T, page_table=t.to(DEV)) for t in tables]

    outs = fresh_outs()
    kvc.kvc_chain(a0, pl, states, rope, outs)
    torch.cuda.synchronize()
    # the first agent's cache is exact: untouched
    assert torch.equal(a0.k.cpu(), a0_cpu.k) and torch.equal(a0.v.cpu(), a0_cpu.v)
    # hop 1 has oracle-identical inputs: strict parity
    _assert_parity(outs[0], orefs[0][0], orefs[0][1], oouts[0])
    # kvc_chain is exactly the sequence of single hops
    step = fresh_outs()
    cur = a0
    for a in range(1, n):
        kvc.kvc_apply(cur, states[a - 1], pl[a] - pl[a - 1], rope, step[a - 1])
        cur = step[a - 1]
    torch.cuda.synchronize()
    for a in range(n - 1):
        assert torch.equal(outs[a].k, step[a].k) and torch.equal(outs[a].v, step[a].v)
    # every later hop, strictly, from the ORACLE's materialised source (oracle -> library only)
    for a in range(2, n):
        o_src = oouts[a - 2]
        src = kvc.Cache(torch.from_numpy(o_src.k.view(np.int16)).view(torch.bfloat16).to(DEV),
                        torch.from_numpy(o_src.v.view(np.int16)).view(torch.bfloat16).to(DEV),
                        T=cfg.T if cfg.paged else None,
                        page_table=None if not cfg.paged else torch.from_numpy(o_src.page_table).to(DEV))
        dst = fresh_outs()[a - 1]
        kvc.kvc_apply(src, states[a - 1], pl[a] - pl[a - 1], rope, dst)
        torch.cuda.synchronize()
        _assert_parity(dst, orefs[a - 1][0], orefs[a - 1][1], oouts[a - 1])
    # end to end the two chains stay together: a rare one-ulp difference at a hop moves the
    # next hop's input by one bf16 step, so the bar here is statistical
    for a in range(n - 1):
        for which, ref in (("k", orefs[a][0]), ("v", orefs[a][1])):
            got = orc.bf16_to_f64(hp.logical_bits(outs[a], which))
            bad = np.abs(got - ref) > hp.BF16_REL * np.abs(ref) + hp.BF16_ABS
            assert bad.mean() < 1e-3
            rown = np.linalg.norm(ref, axis=-1, keepdims=True) + 1e-6
            assert np.max(np.abs(got - ref) / rown) < 2.0 ** -6


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_apply_batch_ragged(path):
    # a small serving batch: per-request length, rank and shift, one shared paged pool each
    reqs = wl.serving_batch(n_requests=7, seed=1, median_T=300, t_lo=40, t_hi=900, ranks=(16, 32, 64))
    kvc.kvc_set_path(path)
    rope = kvc.Rope(500000.0)
    items, singles, oracles = [], [], []
    for i, rq in enumerate(reqs):
        cfg = wl.CONFIGS["llama8b_8k"].scaled(name=f"rq{i}", L=2, H=2, T=rq.T, r=rq.r, paged=(i % 2 == 0), seed=10 + i,
                                               prefix=rq.prefix, n_agents=rq.n_agents, outliers=4)
        src_cpu = hp.make_cache(cfg)
        st_cpu = hp.make_state(cfg, 1, n_cov=rq.T if i != 3 else rq.T // 2)
        shift = rq.prefix[1] - rq.prefix[0]
        src, st = hp.to_dev(src_cpu, DEV), hp.state_to_dev(st_cpu, DEV)
        dst = hp.empty_dst(src_cpu, cfg, DEV, fill=1.0)
        one = hp.empty_dst(src_cpu, cfg, DEV, fill=1.0)
        items.append(kvc.Item(src, dst, st, shift))
        singles.append((src, st, shift, one))
        oracles.append((cfg, src_cpu, st_cpu, shift, dst))
    nb = kvc.kvc_batch_workspace_bytes(len(items))
    ws = torch.empty(nb, dtype=torch.uint8, device=DEV)
    staging = torch.empty(nb, dtype=torch.uint8).pin_memory()
    kvc.kvc_apply_batch(items, rope, ws, staging)
    for (src, st, shift, one) in singles:
        kvc.kvc_apply(src, st, shift, rope, one)
    torch.cuda.synchronize()
    for it, (_, _, _, one), (cfg, src_cpu, st_cpu, shift, dst) in zip(items, singles, oracles):
        assert torch.equal(it.dst.k, one.k) and torch.equal(it.dst.v, one.v)
        odst, ref_k, ref_v = _oracle_hop(cfg, src_cpu, st_cpu, shift,
                                         None if dst.page_table is None else dst.page_table.cpu().numpy())
        _assert_parity(it.dst, ref_k, ref_v, odst)


@pytest.mark.parametrize("cfg", [CFG_VLM_S, CFG_R64_S, CFG_VLM_S.scaled(name="vlm_page32", page=32, T=1999)], ids=lambda c: c.name)
def test_token_major_pages_give_the_same_bits(cfg):
    """A pool whose pages are [page, H, d] (each token with all its heads, the layout of the common paged
    attention kernels) instead of [H, page, d]: the same call, described through the strides, gives the same bits
    in the same logical places - one hop, the fused chain and the multi-anchor apply."""
    rope = kvc.Rope(cfg.theta)
    src_cpu = hp.make_cache(cfg)
    tm = lambda t: t.permute(0, 1, 3, 2, 4).contiguous()
    hm = lambda t: t.permute(0, 1, 3, 2, 4).contiguous()           # its own inverse: swaps the two middle axes back
    src = hp.to_dev(src_cpu, DEV)
    src_t = kvc.Cache(tm(src.k), tm(src.v), T=cfg.T, page_table=src.page_table, token_major=True)
    pl = wl.prefix_lengths(cfg)[:3]
    states = [hp.state_to_dev(hp.make_state(cfg, a), DEV) for a in (1, 2)]
    def dsts(token_major, n):
        out = []
        for a in range(n):
            d = hp.empty_dst(src_cpu, cfg, DEV, table_tag=70 + a, fill=4.0)
            out.append(kvc.Cache(tm(d.k), tm(d.v), T=cfg.T, page_table=d.page_table, token_major=True) if token_major else d)
        return out
    # one hop
    a, b = dsts(False, 1)[0], dsts(True, 1)[0]
    kvc.kvc_apply(src, states[0], pl[1] - pl[0], rope, a)
    kvc.kvc_apply(src_t, states[0], pl[1] - pl[0], rope, b)
    torch.cuda.synchronize()
    assert kvc.kvc_last_path() == kvc.KVC_PATH_TC
    assert torch.equal(hm(b.k), a.k) and torch.equal(hm(b.v), a.v)
    # fused chain (two hops)
    ca, cb = dsts(False, 2), dsts(True, 2)
    ws = torch.empty(max(kvc.kvc_chain_workspace_bytes(src, 3), 128), dtype=torch.uint8, device=DEV)
    kvc.kvc_chain_fused(src, pl, states, rope, ca, ws)
    kvc.kvc_chain_fused(src_t, pl, states, rope, cb, ws)
    torch.cuda.synchronize()
    for x, y in zip(ca, cb):
        assert torch.equal(hm(y.k), x.k) and torch.equal(hm(y.v), x.v)
    assert torch.equal(ca[0].k, a.k)                          # and the chain's first hop is the single hop
    # multi-anchor apply, unit weights
    if cfg.r <= 64:
        ma, mb = dsts(False, 1)[0], dsts(True, 1)[0]
        wsm = torch.empty(max(kvc.kvc_multi_workspace_bytes(src, states), 128), dtype=torch.uint8, device=DEV)
        kvc.kvc_apply_multi(src, states, None, None, 11, rope, ma, wsm)
        kvc.kvc_apply_multi(src_t, states, None, None, 11, rope, mb, wsm)
        torch.cuda.synchronize()
        assert torch.equal(hm(mb.k), ma.k) and torch.equal(hm(mb.v), ma.v)


def test_token_major_contiguous_cache_gives_the_same_bits():
    """A contiguous cache held as [L, T, H, d] instead of [L, H, T, d], through the strides: one hop, the chain
    and a projection give the same bits in the same logical places."""
    cfg = CFG_8B_S
    rope = kvc.Rope(cfg.theta)
    src_cpu = hp.make_cache(cfg)
    src = hp.to_dev(src_cpu, DEV)
    tm = lambda t: t.permute(0, 2, 1, 3).contiguous()
    src_t = kvc.Cache(tm(src.k), tm(src.v), token_major=True)
    pl = wl.prefix_lengths(cfg)[:3]
    states = [hp.state_to_dev(hp.make_state(cfg, a), DEV) for a in (1, 2)]
    outs = [kvc.Cache(torch.zeros_like(src.k), torch.zeros_like(src.v)) for _ in range(2)]
    outs_t = [kvc.Cache(torch.zeros_like(src_t.k), torch.zeros_like(src_t.v), token_major=True) for _ in range(2)]
    kvc.kvc_chain(src, pl, states, rope, outs)
    kvc.kvc_chain(src_t, pl, states, rope, outs_t)
    torch.cuda.synchronize()
    assert kvc.kvc_last_path() == kvc.KVC_PATH_TC
    for a, b in zip(outs, outs_t):
        assert torch.equal(tm(b.k), a.k) and torch.equal(tm(b.v), a.v)
    # projection of the second agent's cache against the first, both layouts
    sts = []
    for s_, t_ in ((src, outs[0]), (src_t, outs_t[0])):
        st = kvc.State(torch.zeros(cfg.L, cfg.H, cfg.T, cfg.r, device=DEV), torch.zeros(cfg.L, cfg.H, cfg.T, cfg.r, device=DEV),
                       states[1].basis_k.clone(), states[1].basis_v.clone())
        kvc.kvc_state_update(s_, t_, pl[1] - pl[0], rope, st, kvc.KVC_PROJECT)
        sts.append(st)
    torch.cuda.synchronize()
    assert torch.equal(sts[0].coeff_k, sts[1].coeff_k) and torch.equal(sts[0].coeff_v, sts[1].coeff_v)
