"""Python binding of the KV-correction CUDA library (``libkvc.so``).

Argument marshalling only: torch tensors supply device memory and the stream,
every step of the path runs in the library's kernels.  The functions carry the
C ABI's names (``include/kvc.h``) and raise :class:`KvcError` on a non-zero
status.  There is no CPU fallback: if the shared object is missing or cannot
be loaded, the first call raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libkvc.so")

KVC_CONTIG, KVC_PAGED = 0, 1
KVC_F32, KVC_BF16 = 0, 1
KVC_ROPE_HALF, KVC_ROPE_INTERLEAVED = 0, 1
KVC_PROJECT, KVC_FIT, KVC_FIT_FAST = 0, 1, 2
(KVC_SOLVER_SUBSPACE, KVC_SOLVER_FULL_RANK, KVC_SOLVER_FULL_DEPENDENT, KVC_SOLVER_FULL_SLOW, KVC_SOLVER_FULL_NO_GAP,
 KVC_SOLVER_FULL_SWEEPS) = (0, -1, 2, 3, 4, 5)
KVC_PATH_AUTO, KVC_PATH_GENERIC, KVC_PATH_TC, KVC_PATH_MIXED = 0, 1, 2, 3
KVC_MAX_SEGMENTS, KVC_COORDS_TARGET, KVC_COORDS_SOURCE = 16, 0, 1
KVC_GROUP_HEAD, KVC_GROUP_LAYER = 0, 1
KVC_FLAG_BAD_PAGE, KVC_FLAG_WAIT_EXPIRED, KVC_FLAG_NOT_CONVERGED = 1, 2, 4
KVC_OK = 0
(KVC_E_INVALID_ARG, KVC_E_SHAPE, KVC_E_UNSUPPORTED, KVC_E_ALIAS, KVC_E_CUDA, KVC_E_WORKSPACE, KVC_E_DEVICE_FLAG,
 KVC_E_TOO_LARGE) = (-1, -2, -3, -4, -5, -6, -7, -8)

EXPORTS = (
    "kvc_apply", "kvc_chain", "kvc_state_update", "kvc_state_update_noalloc", "kvc_workspace_bytes", "kvc_apply_batch",
    "kvc_batch_workspace_bytes", "kvc_status_poll", "kvc_status_reset", "kvc_set_path", "kvc_last_path",
    "kvc_apply_bytes", "kvc_update_bytes", "kvc_strerror", "kvc_version", "kvc_gate_distance", "kvc_gate_weights",
    "kvc_apply_multi", "kvc_multi_workspace_bytes", "kvc_token_weights", "kvc_token_weights_workspace_bytes",
    "kvc_state_realign", "kvc_effective_rank", "kvc_fit_eigenvalues", "kvc_fit_solver", "kvc_group_fit_eigenvalues", "kvc_group_fit_solver", "kvc_selftest_wait_expiry", "kvc_apply_segmented", "kvc_state_update_segmented", "kvc_state_update_check", "kvc_state_update_chain",
    "kvc_chain_update_workspace_bytes", "kvc_chain_update_edge_stride", "kvc_chain_fused", "kvc_chain_workspace_bytes",
)


class KvcError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {strerror(code)} ({code})")
        self.code = code


class kvc_cache(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("layout", C.c_int32), ("L", C.c_int32), ("H", C.c_int32),
                ("T", C.c_int32), ("d", C.c_int32), ("page_size", C.c_int32), ("n_phys_pages", C.c_int32),
                ("page_table", C.c_void_p), ("s_layer", C.c_int64), ("s_page", C.c_int64), ("s_head", C.c_int64),
                ("s_tok", C.c_int64)]


class kvc_state(C.Structure):
    _fields_ = [("coeff_k", C.c_void_p), ("coeff_v", C.c_void_p), ("basis_k", C.c_void_p), ("basis_v", C.c_void_p),
                ("r", C.c_int32), ("n_cov", C.c_int32), ("basis_dtype", C.c_int32), ("grouping", C.c_int32)]


class kvc_rope(C.Structure):
    _fields_ = [("theta", C.c_double), ("pairing", C.c_int32), ("reserved", C.c_int32), ("inv_freq", C.c_void_p)]


class kvc_segments(C.Structure):
    _fields_ = [("n", C.c_int32), ("t_begin", C.POINTER(C.c_int32)), ("shift", C.POINTER(C.c_int32)), ("coords", C.c_int32)]


class kvc_item(C.Structure):
    _fields_ = [("src", kvc_cache), ("dst", kvc_cache), ("st", kvc_state), ("shift", C.c_int32),
                ("t_begin", C.c_int32), ("t_end", C.c_int32), ("reserved", C.c_int32)]


_lib = None


def load(path: Optional[str] = None):
    """Load the shared library (once).  Raises if it is not there: no fallback."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise RuntimeError(f"{p} not found: build it with `python -m paper_2609_34060_b200.build`")
    lib = C.CDLL(p)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    PC, PS, PR, PI = C.POINTER(kvc_cache), C.POINTER(kvc_state), C.POINTER(kvc_rope), C.POINTER(kvc_item)
    lib.kvc_apply.argtypes = [PC, PS, i32, PR, PC, vp]
    lib.kvc_chain.argtypes = [PC, i32, C.POINTER(i32), PS, PR, PC, vp]
    lib.kvc_chain_fused.argtypes = [PC, i32, C.POINTER(i32), PS, PR, PC, vp, sz, vp]
    lib.kvc_chain_workspace_bytes.argtypes = [PC, i32]
    lib.kvc_chain_workspace_bytes.restype = sz
    lib.kvc_state_update.argtypes = [PC, PC, i32, PR, PS, i32, vp, sz, vp]
    lib.kvc_state_update_noalloc.argtypes = [PC, PC, i32, PR, PS, i32, vp]
    lib.kvc_selftest_wait_expiry.argtypes = [C.c_double, C.POINTER(i32), vp]
    PSeg = C.POINTER(kvc_segments)
    lib.kvc_apply_segmented.argtypes = [PC, PS, PSeg, PR, PC, vp]
    lib.kvc_state_update_segmented.argtypes = [PC, PC, PSeg, PR, PS, i32, vp, sz, vp]
    lib.kvc_state_update_check.argtypes = [PC, PC, i32, PR, PS, i32]
    lib.kvc_state_update_chain.argtypes = [PC, i32, C.POINTER(i32), PR, PS, i32, vp, sz, vp]
    lib.kvc_chain_update_workspace_bytes.argtypes = [PC, i32, PS, i32]
    lib.kvc_chain_update_workspace_bytes.restype = sz
    lib.kvc_chain_update_edge_stride.argtypes = [PC, PS, i32]
    lib.kvc_chain_update_edge_stride.restype = sz
    lib.kvc_state_update_noalloc.restype = C.c_int
    lib.kvc_workspace_bytes.argtypes = [PC, PS, i32]
    lib.kvc_workspace_bytes.restype = sz
    lib.kvc_apply_batch.argtypes = [PI, i32, PR, vp, sz, vp, vp]
    lib.kvc_batch_workspace_bytes.argtypes = [i32]
    lib.kvc_batch_workspace_bytes.restype = sz
    lib.kvc_apply_multi.argtypes = [PC, PS, i32, vp, vp, i32, PR, PC, vp, sz, vp]
    lib.kvc_multi_workspace_bytes.argtypes = [PC, PS, i32]
    lib.kvc_multi_workspace_bytes.restype = sz
    lib.kvc_effective_rank.argtypes = [vp, i32, i32, C.c_double, vp, vp]
    lib.kvc_fit_eigenvalues.argtypes = [PC, vp]
    lib.kvc_fit_eigenvalues.restype = vp
    lib.kvc_fit_solver.argtypes = [PC, vp]
    lib.kvc_fit_solver.restype = vp
    lib.kvc_group_fit_eigenvalues.argtypes = [PC, vp]
    lib.kvc_group_fit_eigenvalues.restype = vp
    lib.kvc_group_fit_solver.argtypes = [PC, vp]
    lib.kvc_group_fit_solver.restype = vp
    lib.kvc_state_realign.argtypes = [PS, i32, i32, i32, i32, PR, vp, vp]
    lib.kvc_token_weights.argtypes = [PC, i32, PS, C.POINTER(i32), i32, PR, C.c_double, vp, vp, vp, sz, vp]
    lib.kvc_token_weights_workspace_bytes.argtypes = [PC, i32]
    lib.kvc_token_weights_workspace_bytes.restype = sz
    lib.kvc_gate_distance.argtypes = [PC, PS, i32, i32, vp, vp]
    lib.kvc_gate_weights.argtypes = [vp, i32, C.c_double, vp, vp, vp]
    lib.kvc_status_poll.argtypes = [C.POINTER(C.c_uint32)]
    lib.kvc_status_reset.argtypes = []
    lib.kvc_set_path.argtypes = [i32]
    lib.kvc_last_path.argtypes = []
    lib.kvc_apply_bytes.argtypes = [PC, PS]
    lib.kvc_apply_bytes.restype = i64
    lib.kvc_update_bytes.argtypes = [PC, PS, i32, i32]
    lib.kvc_update_bytes.restype = i64
    lib.kvc_strerror.argtypes = [C.c_int]
    lib.kvc_strerror.restype = C.c_char_p
    lib.kvc_version.argtypes = []
    lib.kvc_version.restype = C.c_char_p
    for name in ("kvc_apply", "kvc_chain", "kvc_state_update", "kvc_apply_batch", "kvc_status_poll",
                 "kvc_status_reset", "kvc_set_path", "kvc_last_path"):
        getattr(lib, name).restype = C.c_int
    if path is None:
        _lib = lib
    return lib


def strerror(code: int) -> str:
    return load().kvc_strerror(code).decode()


def version() -> str:
    return load().kvc_version().decode()


# ---- descriptors over torch tensors ------------------------------------------------


class Cache:
    """A cache descriptor over torch tensors (which it keeps alive).

    contiguous: ``k``, ``v`` bf16 [L, H, T, d]; ``token_major=True``: [L, T, H, d] (each token with all its
                heads), described to the library through the strides.
    paged:      ``k``, ``v`` bf16 pools [L, P, H, page, d], ``page_table`` int32
                [ceil(T/page)], ``T`` the logical length.  ``token_major=True``: the pools
                are [L, P, page, H, d] (a page holds its tokens one after the other, each
                with all heads), described to the library through the strides.
    """

    def __init__(self, k: torch.Tensor, v: torch.Tensor, T: Optional[int] = None,
                 page_table: Optional[torch.Tensor] = None, token_major: bool = False):
        assert k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16
        assert k.is_contiguous() and v.is_contiguous() and k.shape == v.shape
        self.k, self.v, self.page_table = k, v, page_table
        self.token_major = bool(token_major)
        if page_table is None:
            if token_major:
                self.L, self.T, self.H, self.d = (int(x) for x in k.shape)
            else:
                self.L, self.H, self.T, self.d = (int(x) for x in k.shape)
            self.page, self.P = 0, 0
        else:
            assert page_table.dtype == torch.int32 and page_table.is_contiguous() and T is not None
            if token_major:
                self.L, self.P, self.page, self.H, self.d = (int(x) for x in k.shape)
            else:
                self.L, self.P, self.H, self.page, self.d = (int(x) for x in k.shape)
            self.T = int(T)

    def struct(self) -> kvc_cache:
        s = kvc_cache()
        s.k, s.v = self.k.data_ptr(), self.v.data_ptr()
        s.L, s.H, s.T, s.d = self.L, self.H, self.T, self.d
        if self.page_table is None:
            s.layout = KVC_CONTIG
            if self.token_major:
                s.s_tok, s.s_head = self.H * self.d, self.d
                s.s_layer = self.T * self.H * self.d
        else:
            s.layout = KVC_PAGED
            s.page_size, s.n_phys_pages = self.page, self.P
            s.page_table = self.page_table.data_ptr()
            if self.token_major:
                s.s_tok, s.s_head = self.H * self.d, self.d
                s.s_page = self.page * self.H * self.d
                s.s_layer = self.P * s.s_page
        return s

    def empty_like(self, page_table: Optional[torch.Tensor] = None, fill: Optional[float] = None) -> "Cache":
        mk = (lambda t: torch.empty_like(t)) if fill is None else (lambda t: torch.full_like(t, fill))
        if self.page_table is None:
            return Cache(mk(self.k), mk(self.v), token_major=self.token_major)
        return Cache(mk(self.k), mk(self.v), T=self.T,
                     page_table=self.page_table if page_table is None else page_table, token_major=self.token_major)

    def nbytes(self) -> int:
        return self.k.numel() * 2 + self.v.numel() * 2


class State:
    """Rank-r state over torch tensors.  Per (layer, head): coeff fp32 [L,H,n_cov,r], basis fp32|bf16
    [L,H,r,d].  Per layer (``grouping=KVC_GROUP_LAYER``): coeff [L,n_cov,r], basis [L,r,H*d]."""

    def __init__(self, coeff_k, coeff_v, basis_k, basis_v, n_cov: Optional[int] = None, grouping: int = KVC_GROUP_HEAD):
        self.coeff_k, self.coeff_v, self.basis_k, self.basis_v = coeff_k, coeff_v, basis_k, basis_v
        self.grouping = int(grouping)
        g = self.grouping == KVC_GROUP_LAYER
        self.r = 0 if basis_k is None else int(basis_k.shape[1 if g else 2])
        self.n_cov = (0 if coeff_k is None else int(coeff_k.shape[1 if g else 2])) if n_cov is None else int(n_cov)
        if self.r > 0:
            assert basis_k.is_contiguous() and basis_v.is_contiguous() and basis_k.dtype == basis_v.dtype
            assert basis_k.dtype in (torch.float32, torch.bfloat16)
        if self.r > 0 and self.n_cov > 0:
            assert coeff_k.dtype == torch.float32 and coeff_v.dtype == torch.float32
            assert coeff_k.is_contiguous() and coeff_v.is_contiguous()
            assert int(coeff_k.shape[-2]) == self.n_cov and int(coeff_k.shape[-1]) == self.r

    @staticmethod
    def empty() -> "State":
        return State(None, None, None, None, n_cov=0)

    @staticmethod
    def values_only(coeff_v, basis_v) -> "State":
        """Value factors alone (what the reliability gate reads); the key pointers are NULL."""
        s = State.__new__(State)
        s.coeff_k = s.basis_k = None
        s.coeff_v, s.basis_v = coeff_v, basis_v
        s.r, s.n_cov = int(basis_v.shape[2]), int(coeff_v.shape[2])
        assert coeff_v.dtype == torch.float32 and coeff_v.is_contiguous() and basis_v.is_contiguous()
        assert basis_v.dtype in (torch.float32, torch.bfloat16) and int(coeff_v.shape[3]) == s.r
        return s

    # ---- a state as one self-describing blob (header, coefficients, bases): checkpoint / resume of a profiled
    # correction, and the way to keep a failing case.  Host-side plumbing only.
    _BLOB_MAGIC = b"KVCSTATE"

    def dump(self) -> bytes:
        import struct as _st
        parts, meta = [], []
        for t in (self.coeff_k, self.coeff_v, self.basis_k, self.basis_v):
            if t is None:
                meta.append((0, 0, ()))
                continue
            c = t.detach().cpu().contiguous()
            raw = c.view(torch.int16).numpy().tobytes() if c.dtype == torch.bfloat16 else c.numpy().tobytes()
            meta.append((1, 2 if c.dtype == torch.bfloat16 else 4, tuple(int(x) for x in c.shape)))
            parts.append(raw)
        head = self._BLOB_MAGIC + _st.pack("<5i", 1, self.r, self.n_cov, getattr(self, "grouping", KVC_GROUP_HEAD), len(meta))
        for present, esize, shape in meta:
            head += _st.pack("<3i", present, esize, len(shape)) + _st.pack("<%dq" % len(shape), *shape)
        return head + b"".join(parts)

    @staticmethod
    def load(blob: bytes, device="cpu") -> "State":
        import struct as _st
        import numpy as _np
        if blob[:8] != State._BLOB_MAGIC:
            raise ValueError("not a state blob")
        ver, r, n_cov, grouping, n = _st.unpack_from("<5i", blob, 8)
        if ver != 1 or n != 4:
            raise ValueError("unknown state blob version")
        off, meta = 8 + 20, []
        for _ in range(n):
            present, esize, nd = _st.unpack_from("<3i", blob, off)
            off += 12
            shape = _st.unpack_from("<%dq" % nd, blob, off)
            off += 8 * nd
            meta.append((present, esize, shape))
        ts = []
        for present, esize, shape in meta:
            if not present:
                ts.append(None)
                continue
            cnt = 1
            for x in shape:
                cnt *= x
            if esize == 2:
                a = _np.frombuffer(blob, dtype=_np.int16, count=cnt, offset=off).copy()
                t = torch.from_numpy(a).view(torch.bfloat16)
            else:
                a = _np.frombuffer(blob, dtype=_np.float32, count=cnt, offset=off).copy()
                t = torch.from_numpy(a)
            off += cnt * esize
            ts.append(t.reshape(shape).to(device))
        if off != len(blob):
            raise ValueError("state blob has trailing or missing bytes")
        if ts[0] is None and ts[2] is None and ts[3] is not None:
            return State.values_only(ts[1], ts[3])
        return State(ts[0], ts[1], ts[2], ts[3], n_cov=n_cov, grouping=grouping)

    def struct(self) -> kvc_state:
        s = kvc_state()
        ptr = lambda t: 0 if t is None else t.data_ptr()
        s.coeff_k, s.coeff_v, s.basis_k, s.basis_v = ptr(self.coeff_k), ptr(self.coeff_v), ptr(self.basis_k), ptr(self.basis_v)
        s.r, s.n_cov = self.r, self.n_cov
        s.grouping = getattr(self, "grouping", KVC_GROUP_HEAD)
        b = self.basis_k if self.basis_k is not None else self.basis_v
        s.basis_dtype = KVC_BF16 if (b is not None and b.dtype == torch.bfloat16) else KVC_F32
        return s


class Rope:
    def __init__(self, theta: float = 10000.0, pairing: int = KVC_ROPE_HALF, inv_freq: Optional[Sequence[float]] = None):
        self.theta, self.pairing = float(theta), int(pairing)
        self._tab = None if inv_freq is None else (C.c_double * len(inv_freq))(*[float(x) for x in inv_freq])

    def struct(self) -> kvc_rope:
        s = kvc_rope()
        s.theta, s.pairing = self.theta, self.pairing
        s.inv_freq = None if self._tab is None else C.cast(self._tab, C.c_void_p)
        return s


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream) if hasattr(stream, "cuda_stream") else int(stream)


def _check(code: int, what: str):
    if code != 0:
        raise KvcError(code, what)


# ---- the C ABI, same names ---------------------------------------------------------


def kvc_apply(src: Cache, st: State, shift: int, rope: Rope, dst: Cache, stream=None) -> None:
    s, d, t, r = src.struct(), dst.struct(), st.struct(), rope.struct()
    _check(load().kvc_apply(C.byref(s), C.byref(t), int(shift), C.byref(r), C.byref(d), _stream(stream)), "kvc_apply")


def kvc_chain(agent0: Cache, prefix_len: Sequence[int], states: Sequence[State], rope: Rope, outs: Sequence[Cache],
              stream=None) -> None:
    n = len(prefix_len)
    a0, r = agent0.struct(), rope.struct()
    pl = (C.c_int32 * n)(*[int(x) for x in prefix_len])
    sts = (kvc_state * max(n - 1, 1))(*[s.struct() for s in states])
    os_ = (kvc_cache * max(n - 1, 1))(*[o.struct() for o in outs])
    _check(load().kvc_chain(C.byref(a0), n, pl, sts, C.byref(r), os_, _stream(stream)), "kvc_chain")


def kvc_chain_workspace_bytes(agent0: Cache, n_agents: int) -> int:
    a0 = agent0.struct()
    return int(load().kvc_chain_workspace_bytes(C.byref(a0), int(n_agents)))


def kvc_chain_fused(agent0: Cache, prefix_len: Sequence[int], states: Sequence[State], rope: Rope, outs: Sequence[Cache],
                    workspace: torch.Tensor, stream=None) -> None:
    """kvc_chain in one pass over agent 0's cache (same results bit for bit)."""
    n = len(prefix_len)
    a0, r = agent0.struct(), rope.struct()
    pl = (C.c_int32 * n)(*[int(x) for x in prefix_len])
    sts = (kvc_state * max(n - 1, 1))(*[s.struct() for s in states])
    os_ = (kvc_cache * max(n - 1, 1))(*[o.struct() for o in outs])
    _check(load().kvc_chain_fused(C.byref(a0), n, pl, sts, C.byref(r), os_, workspace.data_ptr(),
                                  workspace.numel() * workspace.element_size(), _stream(stream)), "kvc_chain_fused")


class Segments:
    """Piecewise-constant shifts over the token axis: segment j covers t_begin[j] .. t_begin[j+1]-1."""

    def __init__(self, t_begin: Sequence[int], shift: Sequence[int], coords: int = KVC_COORDS_TARGET):
        assert len(t_begin) == len(shift)
        self.t_begin, self.shift, self.coords = [int(x) for x in t_begin], [int(x) for x in shift], int(coords)
        self._tb = (C.c_int32 * len(self.t_begin))(*self.t_begin)
        self._sh = (C.c_int32 * len(self.shift))(*self.shift)

    def struct(self) -> kvc_segments:
        s = kvc_segments()
        s.n, s.t_begin, s.shift, s.coords = len(self.t_begin), self._tb, self._sh, self.coords
        return s


def kvc_apply_segmented(src: Cache, st: State, segs: Segments, rope: Rope, dst: Cache, stream=None) -> None:
    s, d, t, r, g = src.struct(), dst.struct(), st.struct(), rope.struct(), segs.struct()
    _check(load().kvc_apply_segmented(C.byref(s), C.byref(t), C.byref(g), C.byref(r), C.byref(d), _stream(stream)),
           "kvc_apply_segmented")


def kvc_state_update_segmented(src: Optional[Cache], tgt: Cache, segs: Segments, rope: Rope, st: State, mode: int,
                               workspace: Optional[torch.Tensor] = None, stream=None) -> None:
    t, s, r, g = tgt.struct(), st.struct(), rope.struct(), segs.struct()
    sp = None
    if src is not None:
        ss = src.struct()
        sp = C.byref(ss)
    ws_ptr = 0 if workspace is None else workspace.data_ptr()
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().kvc_state_update_segmented(sp, C.byref(t), C.byref(g), C.byref(r), C.byref(s), int(mode), ws_ptr, ws_bytes,
                                             _stream(stream)), "kvc_state_update_segmented")


def kvc_selftest_wait_expiry(limit_ms: float = 1.0, stream=None):
    """(threads whose wait claimed success, abort flag, cycles waited) of a bounded wait made to run out."""
    res = (C.c_int32 * 3)()
    _check(load().kvc_selftest_wait_expiry(float(limit_ms), res, _stream(stream)), "kvc_selftest_wait_expiry")
    return int(res[0]), int(res[1]), int(res[2])


def kvc_chain_update_workspace_bytes(agents: Sequence[Cache], states: Sequence[State], mode: int) -> int:
    n = len(agents)
    ag = (kvc_cache * n)(*[a.struct() for a in agents])
    sts = (kvc_state * max(n - 1, 1))(*[s.struct() for s in states])
    return int(load().kvc_chain_update_workspace_bytes(ag, n, sts, int(mode)))


def kvc_chain_update_edge_stride(tgt: Cache, st: State, mode: int) -> int:
    t, s = tgt.struct(), st.struct()
    return int(load().kvc_chain_update_edge_stride(C.byref(t), C.byref(s), int(mode)))


def kvc_state_update_chain(agents: Sequence[Cache], prefix_len: Sequence[int], rope: Rope, states: Sequence[State],
                           mode: int, workspace: Optional[torch.Tensor] = None, stream=None) -> None:
    """The states of every edge agents[a-1] -> agents[a] in one call (all eigensolves in one launch)."""
    n = len(agents)
    ag = (kvc_cache * n)(*[a.struct() for a in agents])
    pl = (C.c_int32 * n)(*[int(x) for x in prefix_len])
    sts = (kvc_state * max(n - 1, 1))(*[s.struct() for s in states])
    r = rope.struct()
    ws_ptr = 0 if workspace is None else workspace.data_ptr()
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().kvc_state_update_chain(ag, n, pl, C.byref(r), sts, int(mode), ws_ptr, ws_bytes, _stream(stream)),
           "kvc_state_update_chain")


def kvc_workspace_bytes(tgt: Cache, st: State, mode: int) -> int:
    t, s = tgt.struct(), st.struct()
    return int(load().kvc_workspace_bytes(C.byref(t), C.byref(s), int(mode)))


def kvc_state_update(src: Optional[Cache], tgt: Cache, shift: int, rope: Rope, st: State, mode: int,
                     workspace: Optional[torch.Tensor] = None, stream=None) -> None:
    t, s, r = tgt.struct(), st.struct(), rope.struct()
    sp = None
    if src is not None:
        ss = src.struct()
        sp = C.byref(ss)
    ws_ptr = 0 if workspace is None else workspace.data_ptr()
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().kvc_state_update(sp, C.byref(t), int(shift), C.byref(r), C.byref(s), int(mode), ws_ptr, ws_bytes,
                                   _stream(stream)), "kvc_state_update")


KVC_STATIC_SCRATCH_BYTES = 128 * (2 * 128 * 128 + 128) * 4 + 1024


def kvc_state_update_noalloc(src: Optional[Cache], tgt: Cache, shift: int, rope: Rope, st: State, mode: int,
                             stream=None) -> None:
    """kvc_state_update for callers that may not allocate device memory (an engine plugin
    working inside a pre-sized pool, a process whose memory is all committed to the KV
    pool): FIT-mode scratch is a fixed array inside the library, so there is no workspace
    argument.  Raises KvcError(-8) when the problem needs more than
    KVC_STATIC_SCRATCH_BYTES (L*H > 64 at d = 128).  Calls that may overlap on the GPU must
    be serialised by the caller: they share the one array."""
    t, s, r = tgt.struct(), st.struct(), rope.struct()
    sp = None
    if src is not None:
        ss = src.struct()
        sp = C.byref(ss)
    _check(load().kvc_state_update_noalloc(sp, C.byref(t), int(shift), C.byref(r), C.byref(s), int(mode),
                                           _stream(stream)), "kvc_state_update_noalloc")


class Item:
    """One work item of kvc_apply_batch; (t_begin, t_end) = (0, 0) means all rows of the caches."""

    def __init__(self, src: Cache, dst: Cache, st: State, shift: int, t_begin: int = 0, t_end: int = 0):
        self.src, self.dst, self.st, self.shift = src, dst, st, int(shift)
        self.t_begin, self.t_end = int(t_begin), int(t_end)


def kvc_batch_workspace_bytes(n_items: int) -> int:
    return int(load().kvc_batch_workspace_bytes(int(n_items)))


def kvc_apply_batch(items: Sequence[Item], rope: Rope, workspace: torch.Tensor, staging: torch.Tensor,
                    stream=None) -> None:
    n = len(items)
    arr = (kvc_item * max(n, 1))()
    for i, it in enumerate(items):
        arr[i].src, arr[i].dst, arr[i].st, arr[i].shift = it.src.struct(), it.dst.struct(), it.st.struct(), it.shift
        arr[i].t_begin, arr[i].t_end = getattr(it, "t_begin", 0), getattr(it, "t_end", 0)
    r = rope.struct()
    assert staging.device.type == "cpu" and staging.numel() * staging.element_size() >= kvc_batch_workspace_bytes(n)
    _check(load().kvc_apply_batch(arr, n, C.byref(r), workspace.data_ptr(),
                                  workspace.numel() * workspace.element_size(), staging.data_ptr(), _stream(stream)),
           "kvc_apply_batch")


KVC_MULTI_MAX_BLOCKS = 10


def kvc_multi_tpad(T: int) -> int:
    return (int(T) + 127) // 128 * 128


def _state_array(states: Sequence[State]):
    arr = (kvc_state * max(len(states), 1))()
    for i, a in enumerate(states):
        arr[i] = a.struct()
    return arr


def kvc_multi_workspace_bytes(src: Cache, deltas: Sequence[State]) -> int:
    c = src.struct()
    return int(load().kvc_multi_workspace_bytes(C.byref(c), _state_array(deltas), len(deltas)))


def kvc_apply_multi(src: Cache, deltas: Sequence[State], w_k: Optional[torch.Tensor], w_v: Optional[torch.Tensor],
                    shift: int, rope: Rope, dst: Cache, workspace: torch.Tensor, stream=None) -> None:
    """Eq. 8 with token-wise weights [n_anchors, kvc_multi_tpad(T)] fp32 (None: all ones)."""
    cs, cd, r = src.struct(), dst.struct(), rope.struct()
    for w in (w_k, w_v):
        assert w is None or (w.dtype == torch.float32 and w.is_cuda and w.is_contiguous()
                             and tuple(w.shape) == (len(deltas), kvc_multi_tpad(src.T)))
    ptr = lambda t: 0 if t is None else t.data_ptr()
    _check(load().kvc_apply_multi(C.byref(cs), _state_array(deltas), len(deltas), ptr(w_k), ptr(w_v), int(shift),
                                  C.byref(r), C.byref(cd), workspace.data_ptr(),
                                  workspace.numel() * workspace.element_size(), _stream(stream)), "kvc_apply_multi")


KVC_MAX_ANCHORS = 16


def kvc_effective_rank(tgt: Cache, workspace: torch.Tensor, energy: float = 0.9, stream=None) -> torch.Tensor:
    """Effective ranks int32 [L, H, 2] (K, V) from the eigenvalues a FIT update left in `workspace`."""
    c = tgt.struct()
    ev = load().kvc_fit_eigenvalues(C.byref(c), workspace.data_ptr())
    out = torch.empty(tgt.L, tgt.H, 2, dtype=torch.int32, device=workspace.device)
    _check(load().kvc_effective_rank(ev, tgt.L * tgt.H * 2, tgt.d, float(energy), out.data_ptr(), _stream(stream)),
           "kvc_effective_rank")
    return out


def kvc_fit_solver(tgt: Cache, workspace: torch.Tensor) -> torch.Tensor:
    """int32 [L, H, 2] view into the workspace of a KVC_FIT_FAST update: KVC_SOLVER_SUBSPACE (0) where
    the subspace solver served the matrix, else the reason the full eigensolver ran."""
    c = tgt.struct()
    p = load().kvc_fit_solver(C.byref(c), workspace.data_ptr())
    if not p:
        raise KvcError(KVC_E_INVALID_ARG, "kvc_fit_solver")
    off = p - workspace.data_ptr()
    n = tgt.L * tgt.H * 2
    return workspace.view(torch.uint8)[off: off + 4 * n].view(torch.int32).view(tgt.L, tgt.H, 2)


def kvc_group_fit_eigenvalues(tgt: Cache, workspace: torch.Tensor) -> torch.Tensor:
    """float32 [L, 2, H d] view into the workspace of a layer-grouped FIT update."""
    c = tgt.struct()
    p = load().kvc_group_fit_eigenvalues(C.byref(c), workspace.data_ptr())
    if not p:
        raise KvcError(KVC_E_INVALID_ARG, "kvc_group_fit_eigenvalues")
    off = p - workspace.data_ptr()
    n = tgt.L * 2 * tgt.H * tgt.d
    return workspace.view(torch.uint8)[off: off + 4 * n].view(torch.float32).view(tgt.L, 2, tgt.H * tgt.d)


def kvc_group_fit_solver(tgt: Cache, workspace: torch.Tensor) -> torch.Tensor:
    """int32 [L, 2] view into the workspace of a layer-grouped FIT update: 0 where the result was accepted."""
    c = tgt.struct()
    p = load().kvc_group_fit_solver(C.byref(c), workspace.data_ptr())
    if not p:
        raise KvcError(KVC_E_INVALID_ARG, "kvc_group_fit_solver")
    off = p - workspace.data_ptr()
    n = tgt.L * 2
    return workspace.view(torch.uint8)[off: off + 4 * n].view(torch.int32).view(tgt.L, 2)


def kvc_state_realign(st: State, shift: int, rope: Rope, out: Optional[torch.Tensor] = None, stream=None) -> State:
    """A state whose key correction is re-aligned by `shift` positions: basis_k rows rotated (into `out`,
    a new tensor by default; pass st.basis_k for in place); coefficients and value factors are shared."""
    if getattr(st, "grouping", KVC_GROUP_HEAD) == KVC_GROUP_LAYER:
        raise KvcError(KVC_E_UNSUPPORTED, "kvc_state_realign on a per-layer state: pass its geometry through the C call")
    L, H, r, d = (int(x) for x in st.basis_k.shape)
    out = torch.empty_like(st.basis_k) if out is None else out
    s, rp = st.struct(), rope.struct()
    _check(load().kvc_state_realign(C.byref(s), L, H, d, int(shift), C.byref(rp), out.data_ptr(), _stream(stream)),
           "kvc_state_realign")
    return State(st.coeff_k, st.coeff_v, out, st.basis_v, n_cov=st.n_cov)


def kvc_token_weights_workspace_bytes(src: Cache, n_anchors: int) -> int:
    c = src.struct()
    return int(load().kvc_token_weights_workspace_bytes(C.byref(c), int(n_anchors)))


def kvc_token_weights(src: Cache, src_pos: int, anchors: Sequence[State], anchor_pos: Sequence[int], rope: Rope,
                      w_k: torch.Tensor, w_v: torch.Tensor, workspace: torch.Tensor, temperature: float = 1.0,
                      stream=None) -> None:
    """App. A.3 token-wise weights [n_anchors, kvc_multi_tpad(T)] fp32 for keys and for values."""
    n = len(anchors)
    c, r = src.struct(), rope.struct()
    pos = (C.c_int32 * max(n, 1))(*[int(x) for x in anchor_pos])
    for w in (w_k, w_v):
        assert w.dtype == torch.float32 and w.is_cuda and w.is_contiguous() and tuple(w.shape) == (n, kvc_multi_tpad(src.T))
    _check(load().kvc_token_weights(C.byref(c), int(src_pos), _state_array(anchors), pos, n, C.byref(r), float(temperature),
                                    w_k.data_ptr(), w_v.data_ptr(), workspace.data_ptr(),
                                    workspace.numel() * workspace.element_size(), _stream(stream)), "kvc_token_weights")


def kvc_gate_distance(src: Cache, anchors: Sequence[State], k: int, dist_sq: torch.Tensor, stream=None) -> None:
    """Eq. 9, squared: dist_sq[v] (device float64 [len(anchors)]) for every anchor's value factors."""
    n = len(anchors)
    arr = (kvc_state * max(n, 1))()
    for i, a in enumerate(anchors):
        arr[i] = a.struct()
    c = src.struct()
    assert dist_sq.dtype == torch.float64 and dist_sq.is_cuda and dist_sq.numel() >= n
    _check(load().kvc_gate_distance(C.byref(c), arr, n, int(k), dist_sq.data_ptr(), _stream(stream)), "kvc_gate_distance")


def kvc_gate_weights(dist_sq: torch.Tensor, g: torch.Tensor, entropy: torch.Tensor, temperature: float = 1.0,
                     stream=None) -> None:
    """Eqs. 10-11 on the device: g = softmax(-sqrt(dist_sq)/T), entropy[0] = normalised entropy of g."""
    n = int(dist_sq.numel())
    assert dist_sq.dtype == g.dtype == entropy.dtype == torch.float64 and g.numel() >= n and entropy.numel() >= 1
    _check(load().kvc_gate_weights(dist_sq.data_ptr(), n, float(temperature), g.data_ptr(), entropy.data_ptr(),
                                   _stream(stream)), "kvc_gate_weights")


def kvc_status_poll() -> int:
    w = C.c_uint32(0)
    rc = load().kvc_status_poll(C.byref(w))
    if rc not in (0, -7):
        raise KvcError(rc, "kvc_status_poll")
    return int(w.value)


def kvc_status_reset() -> None:
    _check(load().kvc_status_reset(), "kvc_status_reset")


def kvc_set_path(path: int) -> None:
    _check(load().kvc_set_path(int(path)), "kvc_set_path")


def kvc_last_path() -> int:
    return int(load().kvc_last_path())


def kvc_apply_bytes(src: Cache, st: State) -> int:
    s, t = src.struct(), st.struct()
    return int(load().kvc_apply_bytes(C.byref(s), C.byref(t)))


def kvc_update_bytes(tgt: Cache, st: State, mode: int, has_src: bool = True) -> int:
    s, t = tgt.struct(), st.struct()
    return int(load().kvc_update_bytes(C.byref(s), C.byref(t), int(mode), int(bool(has_src))))
