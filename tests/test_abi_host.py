"""Host-only checks of the C ABI: the library builds and loads, exports every symbol the
header declares, and rejects bad arguments before touching a device."""
import ctypes as C
import os
import re

import pytest
import torch

import paper_2609_34060_b200 as kvc
from paper_2609_34060_b200 import build as kbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    kbuild.build()
    return kvc.load()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "kvc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(kvc_[a-z_0-9]+)\s*\(", text)
    return sorted(set(names))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/kvc.h but not exported"
    assert set(names) == set(kvc.EXPORTS)


def test_struct_sizes_match_the_header(lib):
    # 2 pointers + 7 int32 (+pad) + pointer + 4 int64
    assert C.sizeof(kvc.kvc_cache) == 8 + 8 + 7 * 4 + 4 + 8 + 32
    assert C.sizeof(kvc.kvc_state) == 4 * 8 + 4 * 4
    assert C.sizeof(kvc.kvc_rope) == 8 + 4 + 4 + 8
    assert C.sizeof(kvc.kvc_item) == 2 * C.sizeof(kvc.kvc_cache) + C.sizeof(kvc.kvc_state) + 16   # shift, t_begin, t_end, reserved


def _cache(k=0x1000, v=0x100000, L=2, H=2, T=64, d=128, layout=kvc.KVC_CONTIG, **kw):
    c = kvc.kvc_cache()
    c.k, c.v, c.L, c.H, c.T, c.d, c.layout = k, v, L, H, T, d, layout
    for a, b in kw.items():
        setattr(c, a, b)
    return c


def _state(r=8, n_cov=64, ptr=0x4000000):
    s = kvc.kvc_state()
    s.coeff_k, s.coeff_v, s.basis_k, s.basis_v = ptr, ptr + 0x100000, ptr + 0x200000, ptr + 0x300000
    s.r, s.n_cov = r, n_cov
    return s


def _rope(theta=10000.0):
    r = kvc.kvc_rope()
    r.theta = theta
    return r


def test_argument_errors_without_a_device(lib):
    src, dst, st, rope = _cache(), _cache(k=0x2000000, v=0x3000000), _state(), _rope()
    ap = lambda s, t, sh, r, d: lib.kvc_apply(C.byref(s) if s else None, C.byref(t) if t else None, sh,
                                              C.byref(r) if r else None, C.byref(d) if d else None, None)
    assert ap(None, st, 0, rope, dst) == -1
    assert ap(src, None, 0, rope, dst) == -1
    assert ap(src, st, 0, None, dst) == -1
    assert ap(_cache(k=0), st, 0, rope, dst) == -1                     # null buffer
    assert ap(_cache(d=96), st, 0, rope, dst) == -3                    # head dim not built
    assert ap(_cache(k=0x1004), st, 0, rope, dst) == -3                # misaligned rows
    assert ap(src, st, 0, rope, _cache(k=0x2000000, v=0x3000000, T=65)) == -2   # geometry differs
    assert ap(src, _state(n_cov=65), 0, rope, dst) == -2               # covered prefix beyond T
    assert ap(src, _state(r=300), 0, rope, dst) == -3
    assert ap(src, st, 0, _rope(theta=-1.0), dst) == -1
    # partial overlap of contiguous caches
    assert ap(src, st, 0, rope, _cache(k=0x1100, v=0x3000000)) == -4
    # dst K buffer over src V buffer
    assert ap(src, st, 0, rope, _cache(k=0x100000, v=0x3000000)) == -4
    # paged descriptors: page size must be a power of two >= 8, table required
    assert ap(_cache(layout=kvc.KVC_PAGED, page_size=12, n_phys_pages=8, page_table=0x9000), st, 0, rope, dst) == -3
    assert ap(_cache(layout=kvc.KVC_PAGED, page_size=16, n_phys_pages=8, page_table=0), st, 0, rope, dst) == -1
    assert ap(_cache(layout=7), st, 0, rope, dst) == -1


def test_chain_and_update_argument_errors(lib):
    a0, rope = _cache(), _rope()
    pl = (C.c_int32 * 3)(10, 20, 30)
    sts = (kvc.kvc_state * 2)(_state(), _state())
    outs = (kvc.kvc_cache * 2)(_cache(k=0x2000000, v=0x3000000), _cache(k=0x1000, v=0x5000000))
    # second output reuses agent 0's key buffer: the exact cache must never be written
    assert lib.kvc_chain(C.byref(a0), 3, pl, sts, C.byref(rope), outs, None) == -4
    assert lib.kvc_chain(C.byref(a0), 0, pl, sts, C.byref(rope), outs, None) == -1
    assert lib.kvc_chain(C.byref(a0), 1, pl, None, C.byref(rope), None, None) == 0   # a single agent: nothing to do
    tgt, st = _cache(), _state()
    upd = lambda mode, ws, nbytes: lib.kvc_state_update(None, C.byref(tgt), 0, C.byref(rope), C.byref(st), mode, ws, nbytes, None)
    assert upd(5, None, 0) == -1
    assert upd(kvc.KVC_FIT, None, 0) == -6                            # FIT needs scratch
    need = lib.kvc_workspace_bytes(C.byref(tgt), C.byref(st), kvc.KVC_FIT)
    assert need == 2 * 2 * 2 * (2 * 128 * 128 + 128) * 4
    assert lib.kvc_workspace_bytes(C.byref(tgt), C.byref(st), kvc.KVC_PROJECT) == 0
    assert upd(kvc.KVC_FIT, 0x7000100, need - 1) == -6                # too small
    assert upd(kvc.KVC_FIT, 0x7000101, need) == -6                    # misaligned


def test_byte_accounting_and_strings(lib):
    src, st = _cache(L=32, H=8, T=8192, d=128), _state(r=32, n_cov=8192)
    # per (token, layer, head), K and V together: read 4d + 8r, write 4d bytes = 1280 at d=128, r=32
    per_tok = 4 * 128 + 8 * 32 + 4 * 128
    basis = 32 * 8 * 2 * 32 * 128 * 4
    assert lib.kvc_apply_bytes(C.byref(src), C.byref(st)) == 32 * 8 * 8192 * per_tok + basis
    # projection pass: read 8d, write 8r
    assert lib.kvc_update_bytes(C.byref(src), C.byref(st), kvc.KVC_PROJECT, 1) == 32 * 8 * 8192 * (8 * 128 + 8 * 32) + basis
    assert kvc.strerror(0) == "ok" and "alias" in kvc.strerror(-4).lower() or "overlap" in kvc.strerror(-4)
    assert "sm_100a" in kvc.version()
    assert lib.kvc_set_path(9) == -1 and lib.kvc_set_path(kvc.KVC_PATH_AUTO) == 0
    assert lib.kvc_batch_workspace_bytes(0) == 0 and lib.kvc_batch_workspace_bytes(3) > 3 * 600


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(RuntimeError):
        kvc.load(str(tmp_path / "nope.so"))


def test_multi_anchor_and_grouping_argument_errors(lib):
    """The entry points added beside the core path reject bad arguments on the host, before any device work."""
    src, dst, rope = _cache(), _cache(k=0x2000000, v=0x3000000), _rope()
    # grouping: only the two declared values
    bad = _state()
    bad.grouping = 7
    assert lib.kvc_apply(C.byref(src), C.byref(bad), 0, C.byref(rope), C.byref(dst), None) == -1
    grouped = _state()
    grouped.grouping = kvc.KVC_GROUP_LAYER
    # per-layer states: the fit serves ranks up to 32 (and wants its own, larger workspace); the gate and
    # the multi-anchor apply do not serve them
    wide = _state(r=40)
    wide.grouping = kvc.KVC_GROUP_LAYER
    assert lib.kvc_state_update(None, C.byref(src), 0, C.byref(rope), C.byref(wide), kvc.KVC_FIT, 0x7000100, 1 << 30, None) == -3
    need = lib.kvc_workspace_bytes(C.byref(src), C.byref(grouped), kvc.KVC_FIT)
    assert need >= 4 * src.L * 2 * (src.H * src.d) * (1 + 4 * grouped.r)       # eigenvalues + four partial back-projections
    assert lib.kvc_state_update(None, C.byref(src), 0, C.byref(rope), C.byref(grouped), kvc.KVC_FIT, 0x7000100, need - 1, None) == kvc.KVC_E_WORKSPACE
    bad_group = _state()
    bad_group.grouping = 9
    assert lib.kvc_gate_distance(C.byref(src), C.byref(bad_group), 1, 8, 0x8000000, None) == -1
    assert lib.kvc_apply_multi(C.byref(src), C.byref(bad_group), 1, None, None, 0, C.byref(rope), C.byref(dst), 0x9000000, 1 << 30, None) == -1
    # byte accounting of a grouped state: the coefficients are shared by the heads
    big, st = _cache(L=32, H=8, T=8192, d=128), _state(r=32, n_cov=8192)
    st.grouping = kvc.KVC_GROUP_LAYER
    assert lib.kvc_apply_bytes(C.byref(big), C.byref(st)) == 32 * 8 * 8192 * 8 * 128 + 32 * 8192 * 8 * 32 + 32 * 8 * 2 * 32 * 128 * 4
    # gate
    st8 = _state()
    assert lib.kvc_gate_distance(C.byref(src), C.byref(st8), 1, 65, 0x8000000, None) == -2      # k beyond T
    assert lib.kvc_gate_distance(C.byref(src), C.byref(_state(n_cov=10)), 1, 20, 0x8000000, None) == -2   # anchor shorter than k
    assert lib.kvc_gate_distance(C.byref(src), C.byref(st8), 1, 8, 0x8000004, None) == -1       # misaligned float64 output
    assert lib.kvc_gate_distance(C.byref(src), None, 0, 8, None, None) == 0                       # no anchors: nothing to do
    assert lib.kvc_gate_weights(0x8000000, 1, C.c_double(1.0), 0x8000100, 0x8000200, None) == -1  # fewer than two anchors
    assert lib.kvc_gate_weights(0x8000000, 3, C.c_double(0.0), 0x8000100, 0x8000200, None) == -1  # temperature
    # multi-anchor apply: limits and workspace
    many = (kvc.kvc_state * 11)(*[_state() for _ in range(11)])
    assert lib.kvc_apply_multi(C.byref(src), many, 11, None, None, 0, C.byref(rope), C.byref(dst), 0x9000000, 1 << 30, None) == -3
    two = (kvc.kvc_state * 2)(_state(r=32), _state(r=64))
    assert lib.kvc_multi_workspace_bytes(C.byref(src), two, 2) == 3 * 2 * 2 * 2 * 128 * 128      # three rank blocks
    assert lib.kvc_apply_multi(C.byref(src), two, 2, 0x8000004, None, 0, C.byref(rope), C.byref(dst), 0x9000000, 1 << 30, None) == -1
    # token weights
    pos = (C.c_int32 * 2)(0, 0)
    tw = lambda n, ws, nb, pr=rope: lib.kvc_token_weights(C.byref(src), 0, two, pos, n, C.byref(pr), C.c_double(1.0), 0xa000000, 0xb000000, ws, nb, None)
    assert lib.kvc_token_weights_workspace_bytes(C.byref(src), 2) == 2 * 2 * 128 * 4              # T = 64 pads to 128
    assert tw(2, None, 0) == -6
    assert tw(17, 0xc000000, 1 << 20) == -3
    inter = _rope()
    inter.pairing = kvc.KVC_ROPE_INTERLEAVED
    assert tw(2, 0xc000000, 1 << 20, inter) == -3
    # chain workspace, effective rank, realign
    assert lib.kvc_chain_workspace_bytes(C.byref(src), 4) == 3 * 2 * 2 * 2 * 2 * 128 * 128
    assert lib.kvc_chain_workspace_bytes(C.byref(src), 1) == 0
    assert lib.kvc_effective_rank(0x8000000, 4, 128, C.c_double(1.5), 0x8001000, None) == -1
    assert lib.kvc_effective_rank(None, 4, 128, C.c_double(0.9), 0x8001000, None) == -1
    assert lib.kvc_fit_eigenvalues(C.byref(src), None) is None
    assert lib.kvc_state_realign(C.byref(st8), 2, 2, 96, 5, C.byref(rope), 0x8000000, None) == -3
    assert lib.kvc_state_realign(C.byref(st8), 2, 2, 128, 5, C.byref(rope), None, None) == -1


def test_state_blob_round_trip():
    """A state goes to one self-describing blob and back bit for bit (per-head, grouped, bf16 bases, value factors
    only, empty), and a damaged blob is refused."""
    g = torch.Generator().manual_seed(3)
    L, H, T, r, d = 2, 3, 17, 4, 8
    per_head = kvc.State(torch.randn(L, H, T, r, generator=g), torch.randn(L, H, T, r, generator=g),
                         torch.randn(L, H, r, d, generator=g), torch.randn(L, H, r, d, generator=g), n_cov=T)
    grouped = kvc.State(torch.randn(L, T, r, generator=g), torch.randn(L, T, r, generator=g),
                        torch.randn(L, r, H * d, generator=g).bfloat16(), torch.randn(L, r, H * d, generator=g).bfloat16(),
                        grouping=kvc.KVC_GROUP_LAYER)
    values = kvc.State.values_only(torch.randn(L, H, T, r, generator=g), torch.randn(L, H, r, d, generator=g))
    for st in (per_head, grouped, values, kvc.State.empty()):
        back = kvc.State.load(st.dump())
        assert (back.r, back.n_cov, getattr(back, "grouping", 0)) == (st.r, st.n_cov, getattr(st, "grouping", 0))
        for name in ("coeff_k", "coeff_v", "basis_k", "basis_v"):
            a, b = getattr(st, name), getattr(back, name)
            assert (a is None) == (b is None)
            if a is not None:
                assert a.dtype == b.dtype and a.shape == b.shape
                assert torch.equal(a.view(torch.int16) if a.dtype == torch.bfloat16 else a,
                                   b.view(torch.int16) if b.dtype == torch.bfloat16 else b)
    blob = per_head.dump()
    with pytest.raises(ValueError):
        kvc.State.load(b"XXXXXXXX" + blob[8:])
    with pytest.raises(ValueError):
        kvc.State.load(blob[:-4])
