"""fp64 CPU oracle for the low-rank KV-cache correction path.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the
CUDA library is checked against.  It shares no code with the CUDA path and the
product never imports it: only the tests, the smoke check and the benchmark's
CPU-baseline leg may call it.

Everything is numpy in float64.  Caches are held as bf16 *bit patterns*
(uint16) exactly as they sit in device memory; they are widened exactly to
float64 before any arithmetic and rounded once, to nearest-even, when a
corrected cache is materialised.

What each function follows in the paper:

* ``rope_shift``      -- the deterministic key re-alignment that every method
                         applies before cross-agent reuse (Sec. 2.2; App. A.2,
                         A.3 "Correction Weighting and Positional Alignment":
                         keys are re-rotated, values need no rotation).
* ``deviation``       -- Eq. 12 (observed transition): Delta = C_j - Align(C_i);
                         Eq. 6 (chained delta).
* ``fit_basis``       -- Eq. 7: truncated SVD Z ~= A_Z B_Z with
                         A = U_r Sigma_r, B = R_r^T (largest r singular values).
* ``project``         -- A = Delta B^T for a given orthonormal-row basis B.
* ``apply``           -- Eq. 8 with one anchor (w = 1): C_hat_j = Align(C_i) +
                         A B, materialised in full dimension (Sec. 3.3);
                         partial coverage per App. A.3 "Variable Segment
                         Lengths" (rows beyond the covered prefix keep the
                         re-aligned source).
* ``chain``           -- Sec. 3.2 / App. A.3 "Cache Materialization": the first
                         agent's cache is exact and never written; each
                         materialised cache is the source of the next edge.
* ``multi_anchor_*``  -- Eq. 8 with V anchors and Eqs. 9-11 (reliability gate).

Parity pins (tests/test_oracle_*.py) tie these to facts fixed outside this
file: a library SVD, closed forms, brute-force loops, the paper's memory
example.  The paper's accuracy / TTFT tables need models and datasets and are
"parity unpinned" here: nothing in this file claims them.
"""
from __future__ import annotations

import numpy as np

# --------------------------------------------------------------------------
# bf16 codec (round-to-nearest-even, one rounding straight from float64)
# --------------------------------------------------------------------------


def bf16_to_f64(bits):
    """Widen bf16 bit patterns (uint16) exactly to float64."""
    b = np.asarray(bits, dtype=np.uint16)
    with np.errstate(invalid="ignore"):               # signalling-NaN patterns widen quietly
        return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def round_to_bf16(x):
    """Round float64 to the nearest bf16 value (ties to even); result is float64.

    bf16 keeps 8 significant bits with the float32 exponent range: normal
    numbers down to 2^-126, a fixed quantum 2^-133 below that, overflow to inf
    from 2^128 on.
    """
    x = np.asarray(x, dtype=np.float64)
    finite = np.isfinite(x)
    xs = np.where(finite, x, 0.0)
    _, e = np.frexp(xs)                       # xs = m * 2**e with 0.5 <= |m| < 1
    e = np.maximum(e, -125)                   # subnormal range: fixed quantum
    q = np.ldexp(1.0, e - 8)                  # spacing of bf16 numbers around xs
    y = np.rint(xs / q) * q                   # np.rint rounds half to even
    y = np.where(np.abs(y) >= 2.0 ** 128, np.copysign(np.inf, xs), y)
    return np.where(finite, y, x)


def f64_to_bf16_bits(x):
    """float64 -> bf16 bit pattern (uint16), one round-to-nearest-even."""
    y = round_to_bf16(x)
    with np.errstate(over="ignore", invalid="ignore"):
        f = y.astype(np.float32)              # exact: y is representable
    return (f.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


# --------------------------------------------------------------------------
# RoPE re-alignment
# --------------------------------------------------------------------------

ROPE_HALF = 0          # channel k pairs with k + d/2
ROPE_INTERLEAVED = 1   # channel 2k pairs with 2k + 1


def rope_inv_freq(d, theta):
    """f_k = theta^(-2k/d), k = 0 .. d/2-1, in float64."""
    k = np.arange(d // 2, dtype=np.float64)
    return np.power(np.float64(theta), -2.0 * k / np.float64(d))


def rope_shift(x, s, inv_freq, pairing=ROPE_HALF):
    """Rotate every channel pair of x[..., d] by the angle s * f_k.

    A cached key written at position p and re-used at position p + s is
    Rot_s of the cached vector; rotations of one pair commute, so only the
    shift matters.  s == 0 returns x itself (no arithmetic).
    """
    if s == 0:
        return x
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    a = np.float64(s) * np.asarray(inv_freq, dtype=np.float64)
    c, sn = np.cos(a), np.sin(a)
    y = np.empty_like(x)
    if pairing == ROPE_HALF:
        x1, x2 = x[..., : d // 2], x[..., d // 2:]
        y[..., : d // 2] = x1 * c - x2 * sn
        y[..., d // 2:] = x1 * sn + x2 * c
    else:
        x1, x2 = x[..., 0::2], x[..., 1::2]
        y[..., 0::2] = x1 * c - x2 * sn
        y[..., 1::2] = x1 * sn + x2 * c
    return y


# --------------------------------------------------------------------------
# Cache containers: contiguous [L,H,T,d] or paged pool [L,P,H,page,d]
# --------------------------------------------------------------------------


class Cache:
    """One agent's shared-context cache as bf16 bit patterns.

    contiguous: ``k``/``v`` are uint16 [L, H, T, d].
    paged:      ``k``/``v`` are uint16 pools [L, P, H, page, d] and logical
                token t of every layer and head lives in physical page
                ``page_table[t // page]`` at row ``t % page``.
    """

    def __init__(self, k, v, T=None, page_table=None):
        self.k = np.asarray(k, dtype=np.uint16)
        self.v = np.asarray(v, dtype=np.uint16)
        assert self.k.shape == self.v.shape
        self.page_table = None if page_table is None else np.asarray(page_table, dtype=np.int32)
        if self.page_table is None:
            assert self.k.ndim == 4
            self.L, self.H, self.T, self.d = self.k.shape
            self.page = 0
        else:
            assert self.k.ndim == 5 and T is not None
            self.L, self.P, self.H, self.page, self.d = self.k.shape
            self.T = int(T)
            assert self.page_table.shape[0] * self.page >= self.T

    def _rows(self):
        t = np.arange(self.T)
        return self.page_table[t // self.page].astype(np.int64), t % self.page

    def get_bits(self, which, l, h):
        """[T, d] uint16 view/copy of one (layer, head) slab in logical order."""
        a = self.k if which == "k" else self.v
        if self.page_table is None:
            return a[l, h]
        p, o = self._rows()
        return a[l, p, h, o, :]

    def put_bits(self, which, l, h, bits):
        a = self.k if which == "k" else self.v
        if self.page_table is None:
            a[l, h] = bits
        else:
            p, o = self._rows()
            a[l, p, h, o, :] = bits

    def empty_like(self, page_table=None, fill=0):
        """A destination cache of the same geometry (optionally another table)."""
        k = np.full_like(self.k, fill)
        v = np.full_like(self.v, fill)
        if self.page_table is None:
            return Cache(k, v)
        pt = self.page_table if page_table is None else page_table
        return Cache(k, v, T=self.T, page_table=pt)


class State:
    """Rank-r state of one hop: coeff fp32 [L,H,n_cov,r], basis [L,H,r,d] (K and V)."""

    def __init__(self, coeff_k, coeff_v, basis_k, basis_v, n_cov=None):
        self.coeff_k = np.asarray(coeff_k)
        self.coeff_v = np.asarray(coeff_v)
        self.basis_k = np.asarray(basis_k)
        self.basis_v = np.asarray(basis_v)
        self.r = int(self.basis_k.shape[2]) if self.basis_k.ndim == 4 else 0
        self.n_cov = int(self.coeff_k.shape[2]) if n_cov is None else int(n_cov)


# --------------------------------------------------------------------------
# apply / chain  (Eq. 8 with one anchor; Sec. 3.2)
# --------------------------------------------------------------------------


def apply_slab(src_bits, coeff, basis, s, inv_freq, n_cov, is_key, pairing=ROPE_HALF):
    """One (layer, head) slab of one hop.

    src_bits [T,d] uint16, coeff [>=n_cov, r], basis [r, d].
    Returns (ref, out_bits): ref is the float64 value before rounding, out_bits
    the materialised bf16 cache.  Rows t >= n_cov (or r == 0) keep the aligned
    source: values, and keys at shift 0, pass through bit for bit.
    """
    x = bf16_to_f64(src_bits)
    T = x.shape[0]
    shift = s if is_key else 0
    aligned = rope_shift(x, shift, inv_freq, pairing)
    ref = np.array(aligned, dtype=np.float64, copy=True)
    r = 0 if basis is None else int(np.asarray(basis).shape[0])
    n = min(int(n_cov), T) if r > 0 else 0
    if n > 0:
        c = np.asarray(coeff[:n], dtype=np.float64)
        b = np.asarray(basis, dtype=np.float64)
        ref[:n] = aligned[:n] + c @ b
    out = f64_to_bf16_bits(ref)
    if shift == 0:
        out[n:] = src_bits[n:]               # nothing computed: bits survive
    return ref, out


def apply(src, st, s, inv_freq, dst=None, pairing=ROPE_HALF, want_ref=False):
    """C_hat = Align_s(src) + coeff @ basis, per (layer, head), K and V."""
    dst = src.empty_like() if dst is None else dst
    refs = {"k": [], "v": []}
    for l in range(src.L):
        for h in range(src.H):
            for which, cf, bs in (("k", st.coeff_k, st.basis_k), ("v", st.coeff_v, st.basis_v)):
                has = st.r > 0 and st.n_cov > 0
                ref, out = apply_slab(
                    src.get_bits(which, l, h),
                    cf[l, h] if has else None,
                    bs[l, h] if has else None,
                    s, inv_freq, st.n_cov if has else 0, which == "k", pairing)
                dst.put_bits(which, l, h, out)
                if want_ref:
                    refs[which].append(ref)
    if want_ref:
        shp = (src.L, src.H, src.T, src.d)
        return dst, np.asarray(refs["k"]).reshape(shp), np.asarray(refs["v"]).reshape(shp)
    return dst


def chain(agent0, prefix_len, states, inv_freq, dst_tables=None, pairing=ROPE_HALF, want_ref=False):
    """Agents 1..N-1 from agent 0 along the workflow.

    Hop a re-aligns by prefix_len[a] - prefix_len[a-1] and applies states[a-1]
    to the *materialised* (bf16) cache of agent a-1.  agent0 is only read.
    Returns the list of N-1 caches (and, on request, each hop's float64
    pre-rounding values).
    """
    outs, refs = [], []
    cur = agent0
    for a in range(1, len(prefix_len)):
        s = int(prefix_len[a]) - int(prefix_len[a - 1])
        dst = cur.empty_like(None if dst_tables is None else dst_tables[a - 1])
        res = apply(cur, states[a - 1], s, inv_freq, dst=dst, pairing=pairing, want_ref=want_ref)
        if want_ref:
            dst, rk, rv = res
            refs.append((rk, rv))
        outs.append(dst)
        cur = dst
    return (outs, refs) if want_ref else outs


def make_target(src, st, s, inv_freq, noise_k, noise_v, sigma, dst=None, pairing=ROPE_HALF):
    """The true cache of the next agent in the synthetic workloads: the re-aligned source
    plus an exactly rank-r deviation plus Gaussian noise, rounded once to bf16:
        C_j = bf16(Align_s(C_i) + A B + sigma * noise).
    noise_* are standard-normal draws [L,H,T,d] handed in by the input generator."""
    dst = src.empty_like() if dst is None else dst
    for l in range(src.L):
        for h in range(src.H):
            for which, cf, bs, nz in (("k", st.coeff_k, st.basis_k, noise_k), ("v", st.coeff_v, st.basis_v, noise_v)):
                ref, _ = apply_slab(src.get_bits(which, l, h), cf[l, h], bs[l, h], s, inv_freq, st.n_cov,
                                    which == "k", pairing)
                dst.put_bits(which, l, h, f64_to_bf16_bits(ref + sigma * np.asarray(nz[l, h], np.float64)))
    return dst


def chain_unrounded_slab(x0, prefix_len, coeffs, bases, inv_freq, is_key, pairing=ROPE_HALF):
    """The same recursion carried in float64 with no intermediate rounding.

    Only for the algebraic pins (closed form by linearity, Eq. 6 equivalence).
    x0 [T,d] float64; coeffs[a-1] [T,r]; bases[a-1] [r,d].  Returns the list of
    float64 caches of agents 1..N-1.
    """
    cur = np.asarray(x0, dtype=np.float64)
    outs = []
    for a in range(1, len(prefix_len)):
        s = (int(prefix_len[a]) - int(prefix_len[a - 1])) if is_key else 0
        cur = rope_shift(cur, s, inv_freq, pairing) + np.asarray(coeffs[a - 1], np.float64) @ np.asarray(bases[a - 1], np.float64)
        outs.append(cur)
    return outs


# --------------------------------------------------------------------------
# state update  (Eq. 12 deviation, Eq. 7 factorisation)
# --------------------------------------------------------------------------


def deviation(src_bits, tgt_bits, s, inv_freq, is_key, pairing=ROPE_HALF):
    """Delta = C_tgt - Align_s(C_src); src_bits None => Delta = C_tgt (base factorisation)."""
    tgt = bf16_to_f64(tgt_bits)
    if src_bits is None:
        return tgt
    src = bf16_to_f64(src_bits)
    return tgt - rope_shift(src, s if is_key else 0, inv_freq, pairing)


def gram(delta):
    """G = Delta^T Delta (d x d)."""
    delta = np.asarray(delta, dtype=np.float64)
    return delta.T @ delta


def jacobi_eigh(G, tol=1e-30, max_sweeps=60):
    """Cyclic Jacobi for a real symmetric matrix.  Returns (eigenvalues, eigenvectors
    as columns), unsorted.  Plain textbook rotations in float64."""
    A = np.array(G, dtype=np.float64, copy=True)
    n = A.shape[0]
    V = np.eye(n)
    scale = max(float(np.sum(A * A)), np.finfo(np.float64).tiny)
    for _ in range(max_sweeps):
        O = A - np.diag(np.diag(A))
        off = float(np.sum(O * O))                    # off-diagonal energy, summed directly
        if off <= tol * scale:
            break
        for p in range(n - 1):
            for q in range(p + 1, n):
                apq = A[p, q]
                if apq == 0.0:
                    continue
                tau = (A[q, q] - A[p, p]) / (2.0 * apq)
                t = (1.0 if tau >= 0 else -1.0) / (abs(tau) + np.sqrt(1.0 + tau * tau))
                c = 1.0 / np.sqrt(1.0 + t * t)
                sn = t * c
                # A <- J^T A J on rows/columns p, q
                Ap, Aq = A[:, p].copy(), A[:, q].copy()
                A[:, p] = c * Ap - sn * Aq
                A[:, q] = sn * Ap + c * Aq
                Ap, Aq = A[p, :].copy(), A[q, :].copy()
                A[p, :] = c * Ap - sn * Aq
                A[q, :] = sn * Ap + c * Aq
                Vp, Vq = V[:, p].copy(), V[:, q].copy()
                V[:, p] = c * Vp - sn * Vq
                V[:, q] = sn * Vp + c * Vq
    return np.diag(A).copy(), V


def fit_basis(delta, r):
    """Top-r right singular vectors of Delta as rows (B = R_r^T of Eq. 7), from the
    eigenvectors of G = Delta^T Delta.  Returns (basis [r,d], eigenvalues [d] sorted
    descending).  Rows beyond min(r, d, T) or with a non-positive eigenvalue are zero.
    Sign convention: the largest-magnitude component of each row is positive."""
    delta = np.asarray(delta, dtype=np.float64)
    T, d = delta.shape
    w, V = jacobi_eigh(gram(delta))
    order = np.argsort(-w, kind="stable")
    w, V = w[order], V[:, order]
    B = np.zeros((r, d))
    for q in range(min(r, d, T)):
        if w[q] <= 0.0:
            continue
        v = V[:, q] / np.linalg.norm(V[:, q])
        if v[int(np.argmax(np.abs(v)))] < 0:
            v = -v
        B[q] = v
    return B, w


def project(delta, basis):
    """A = Delta B^T  (= U_r Sigma_r when B holds the top-r right singular vectors)."""
    return np.asarray(delta, np.float64) @ np.asarray(basis, np.float64).T


FIT, PROJECT = 1, 0


def state_update(src, tgt, s, inv_freq, r=None, mode=PROJECT, basis_k=None, basis_v=None,
                 n_cov=None, pairing=ROPE_HALF):
    """Rank-r state of the edge src -> tgt for every (layer, head), K and V.

    PROJECT: the bases are given, only the coefficients are computed.
    FIT:     bases from Eq. 7, then the coefficients.
    Coefficients are stored as float32 (the state's storage type); bases float32.
    Returns (State, eigenvalues or None) with eigenvalues [L,H,2,d].
    """
    L, H, T, d = tgt.L, tgt.H, tgt.T, tgt.d
    n = T if n_cov is None else int(n_cov)
    if mode == PROJECT:
        r = int(np.asarray(basis_k).shape[2])
    ck = np.zeros((L, H, n, r), np.float32)
    cv = np.zeros((L, H, n, r), np.float32)
    bk = np.zeros((L, H, r, d), np.float32)
    bv = np.zeros((L, H, r, d), np.float32)
    ev = np.zeros((L, H, 2, d)) if mode == FIT else None
    for l in range(L):
        for h in range(H):
            for i, (which, cf, bs, given) in enumerate((("k", ck, bk, basis_k), ("v", cv, bv, basis_v))):
                dlt = deviation(None if src is None else src.get_bits(which, l, h),
                                tgt.get_bits(which, l, h), s, inv_freq, which == "k", pairing)[:n]
                if mode == FIT:
                    B, w = fit_basis(dlt, r)
                    B = B.astype(np.float32)          # the stored basis is what projects
                    ev[l, h, i] = w
                else:
                    B = np.asarray(given[l, h])
                bs[l, h] = B
                cf[l, h] = project(dlt, B).astype(np.float32)
    return State(ck, cv, bk, bv, n_cov=n), ev


# --------------------------------------------------------------------------
# multi-anchor estimate and reliability gate (Eqs. 8-11)
# --------------------------------------------------------------------------


def gate_distance(v_src_layers, v_anchor_layers, k):
    """Eq. 9: sqrt(sum over layers of ||V_src[:k] - V_anchor[:k]||_F^2).
    Each argument is a list over layers of float64 [T, D] matrices."""
    acc = 0.0
    for a, b in zip(v_src_layers, v_anchor_layers):
        diff = np.asarray(a, np.float64)[:k] - np.asarray(b, np.float64)[:k]
        acc += float(np.sum(diff * diff))
    return np.sqrt(acc)


def gate_weights(dist, temperature=1.0):
    """Eq. 10: softmax of -d/T over the compatible anchors."""
    z = -np.asarray(dist, np.float64) / temperature
    z = z - np.max(z)
    e = np.exp(z)
    return e / np.sum(e)


def normalized_entropy(g):
    """Eq. 11: -sum g log2 g / log2 |A_k|  (0 log 0 = 0).  Needs |A_k| >= 2."""
    g = np.asarray(g, np.float64)
    n = g.shape[0]
    if n < 2:
        raise ValueError("fewer than two compatible anchors: dense prefill, no gate value")
    nz = g[g > 0]
    return float(-np.sum(nz * np.log2(nz)) / np.log2(n))


def multi_anchor_delta(weights, coeffs, bases):
    """Eq. 8: sum_v w_v A_v B_v with token-wise weights [V, T] (each column sums to 1)."""
    out = 0.0
    for w, A, B in zip(weights, coeffs, bases):
        out = out + np.asarray(w, np.float64)[:, None] * (np.asarray(A, np.float64) @ np.asarray(B, np.float64))
    return out


def stack_anchors(weights, coeffs, bases):
    """The same estimate as one rank-(V r) state: coeff' = [w_0 A_0 | w_1 A_1 | ...],
    basis' = [B_0; B_1; ...] -- the form the apply kernel consumes."""
    c = np.concatenate([np.asarray(w, np.float64)[:, None] * np.asarray(A, np.float64)
                        for w, A in zip(weights, coeffs)], axis=1)
    b = np.concatenate([np.asarray(B, np.float64) for B in bases], axis=0)
    return c, b


def effective_rank(eigenvalues, energy=0.9):
    """Sec. 3.1 (figure on effective rank): the minimum rank that retains `energy` (90 %) of the
    singular-value energy, the energy of a matrix being the sum of its squared singular values =
    the sum of the eigenvalues of its Gram matrix.  eigenvalues: 1-D, any order, negatives (rounding)
    count as zero.  A zero matrix has effective rank 0."""
    w = np.sort(np.clip(np.asarray(eigenvalues, np.float64), 0.0, None))[::-1]
    total = float(np.sum(w))
    if total <= 0.0:
        return 0
    acc = np.cumsum(w)
    return int(np.searchsorted(acc, energy * total, side="left") + 1)


def ungroup_state(coeff_k, coeff_v, basis_k, basis_v, H, n_cov=None):
    """Sec. 3.1 with D = H d (one state per layer over all KV heads): coeff [L, n_cov, r] is shared by
    the heads of a layer and basis [L, r, H d] holds head h's part in columns h d .. (h+1) d - 1.
    Returns the same state in the per-(layer, head) form, coeff [L, H, n_cov, r] and basis
    [L, H, r, d], which every other function of this module takes: the two forms define the same
    low-rank product  Z[l] = coeff[l] @ basis[l]  with Z[l] = [Z[l,0] | ... | Z[l,H-1]]."""
    ck, cv = np.asarray(coeff_k), np.asarray(coeff_v)
    bk, bv = np.asarray(basis_k), np.asarray(basis_v)
    L, r, HD = bk.shape
    d = HD // H
    split = lambda b: np.ascontiguousarray(b.reshape(L, r, H, d).transpose(0, 2, 1, 3))
    rep = lambda c: np.ascontiguousarray(np.broadcast_to(c[:, None], (L, H) + c.shape[1:]))
    return State(rep(ck), rep(cv), split(bk), split(bv), n_cov=n_cov)


def project_grouped(delta_slabs, basis_l):
    """Projection for one layer under D = H d: delta_slabs is the list over heads of [T, d]
    deviations, basis_l [r, H d]; the coefficients are those of the concatenated deviation
    [T, H d], i.e. the sum over heads of each head's projection on its own columns."""
    cat = np.concatenate([np.asarray(x, np.float64) for x in delta_slabs], axis=1)
    return cat @ np.asarray(basis_l, np.float64).T


def fit_grouped(delta_slabs, r):
    """Eq. 7 for one layer under D = H d (Sec. 3.1): the truncated SVD of the concatenated deviation
    [T, H d] (the heads' deviations side by side on the feature axis).  delta_slabs: list over heads
    of [T, d].  Returns (basis [r, H d], eigenvalues [H d] of its Gram matrix, descending), exactly
    fit_basis on the concatenation."""
    cat = np.concatenate([np.asarray(x, np.float64) for x in delta_slabs], axis=1)
    return fit_basis(cat, r)


# --------------------------------------------------------------------------
# Multi-segment contexts (Eq. 1): a trajectory interleaves agent-specific pieces with the shared ones,
# so the shared tokens of two agents differ by a shift that is constant inside a segment and changes
# from segment to segment.
# --------------------------------------------------------------------------
COORDS_TARGET = 0   # the correction lives at the target's positions: C_hat = Rot_s(src) + c . B      (Eq. 12)
COORDS_SOURCE = 1   # the correction lives at the source's positions: C_hat = Rot_s(src + c . B)      (App. A.2)


def segment_shifts(T, t_begin, shift):
    """Per-token shift vector [T] of a piecewise-constant shift: segment j covers tokens
    t_begin[j] .. t_begin[j+1] - 1 (the last one runs to T) and is shifted by shift[j]."""
    t_begin, shift = list(t_begin), list(shift)
    assert len(t_begin) == len(shift) and (not t_begin or t_begin[0] == 0)
    out = np.zeros(T, dtype=np.int64)
    for j, t0 in enumerate(t_begin):
        t1 = t_begin[j + 1] if j + 1 < len(t_begin) else T
        assert t0 <= t1
        out[t0:t1] = shift[j]
    return out


def rope_shift_tokens(x, s_tok, inv_freq, pairing=ROPE_HALF):
    """rope_shift with one shift per token: row t of x [T, d] is rotated by s_tok[t] * f_k.
    Rows whose shift is 0 are returned untouched."""
    x = np.asarray(x, dtype=np.float64)
    s_tok = np.asarray(s_tok, dtype=np.int64)
    T, d = x.shape
    a = s_tok.astype(np.float64)[:, None] * np.asarray(inv_freq, dtype=np.float64)[None, :]   # [T, d/2]
    c, sn = np.cos(a), np.sin(a)
    y = np.empty_like(x)
    if pairing == ROPE_HALF:
        x1, x2 = x[:, : d // 2], x[:, d // 2:]
        y[:, : d // 2] = x1 * c - x2 * sn
        y[:, d // 2:] = x1 * sn + x2 * c
    else:
        x1, x2 = x[:, 0::2], x[:, 1::2]
        y[:, 0::2] = x1 * c - x2 * sn
        y[:, 1::2] = x1 * sn + x2 * c
    still = s_tok == 0
    y[still] = x[still]
    return y


def apply_slab_tokens(src_bits, coeff, basis, s_tok, inv_freq, n_cov, is_key, pairing=ROPE_HALF, coords=COORDS_TARGET):
    """apply_slab with a per-token shift vector and the choice of the correction's coordinates.
    TARGET: ref = Rot_s(src) + c . B;  SOURCE: ref = Rot_s(src + c . B).  Values are never rotated, so
    for them the two agree.  Rows that are neither covered nor shifted keep their bits."""
    x = bf16_to_f64(src_bits)
    T = x.shape[0]
    s_tok = np.asarray(s_tok, dtype=np.int64) if is_key else np.zeros(T, dtype=np.int64)
    r = 0 if basis is None else int(np.asarray(basis).shape[0])
    n = min(int(n_cov), T) if r > 0 else 0
    corr = np.zeros_like(x)
    if n > 0:
        corr[:n] = np.asarray(coeff[:n], dtype=np.float64) @ np.asarray(basis, dtype=np.float64)
    if coords == COORDS_SOURCE:
        ref = rope_shift_tokens(x + corr, s_tok, inv_freq, pairing)
    else:
        ref = rope_shift_tokens(x, s_tok, inv_freq, pairing) + corr
    out = f64_to_bf16_bits(ref)
    keep = (s_tok == 0) & (np.arange(T) >= n)
    out[keep] = src_bits[keep]
    return ref, out


def deviation_tokens(src_bits, tgt_bits, s_tok, inv_freq, is_key, pairing=ROPE_HALF, coords=COORDS_TARGET):
    """The deviation a state is fitted to, with per-token shifts.  TARGET: tgt - Rot_s(src) (Eq. 12);
    SOURCE: Rot_{-s}(tgt) - src, the same deviation carried back to the source's positions."""
    tgt = bf16_to_f64(tgt_bits)
    if src_bits is None:
        return tgt
    src = bf16_to_f64(src_bits)
    T = src.shape[0]
    s_tok = np.asarray(s_tok, dtype=np.int64) if is_key else np.zeros(T, dtype=np.int64)
    if coords == COORDS_SOURCE:
        return rope_shift_tokens(tgt, -s_tok, inv_freq, pairing) - src
    return tgt - rope_shift_tokens(src, s_tok, inv_freq, pairing)


def realign_basis(basis_k, s, inv_freq, pairing=ROPE_HALF):
    """App. A.2 (PF-induced deltas): a stored key correction is "positionally re-aligned when reused".
    A rotation acts on the channel axis and is linear, so Rot_s(c . B) = c . Rot_s(B): re-aligning a
    stored correction by s positions is rotating every key-basis row by s; coefficients and value
    factors are untouched.  basis_k [..., r, d] -> same shape, float64."""
    b = np.asarray(basis_k, np.float64)
    return rope_shift(b.reshape(-1, b.shape[-1]), s, inv_freq, pairing).reshape(b.shape)


def token_weights(src_feat, anchor_feats, temperature=1.0):
    """App. A.3 "Correction Weighting": token-wise interpolation weights.  For token t and anchor v the
    score is the mean absolute difference between the source cache's features of t and the anchor's
    reconstructed base features of t (mean over all layers, heads and channels); the weights are the
    softmax over anchors of minus the score (T = 1).  Keys and values are weighted separately: call
    once with key features (both sides in canonical positional coordinates) and once with value
    features.  src_feat [T, F]; anchor_feats list over anchors of [T, F].  Returns [V, T]."""
    x = np.asarray(src_feat, np.float64)
    m = np.stack([np.mean(np.abs(x - np.asarray(a, np.float64)), axis=1) for a in anchor_feats])   # [V, T]
    z = -m / temperature
    z = z - np.max(z, axis=0, keepdims=True)
    e = np.exp(z)
    return e / np.sum(e, axis=0, keepdims=True)


def canonical_key_features(bits_slabs, pos, inv_freq, pairing=ROPE_HALF):
    """Keys of one cache in canonical positional coordinates: every (layer, head) slab [T, d] rotated
    back by the cache's own position offset `pos`, slabs concatenated along the feature axis."""
    return np.concatenate([rope_shift(bf16_to_f64(b) if b.dtype == np.uint16 else np.asarray(b, np.float64),
                                      -pos, inv_freq, pairing) for b in bits_slabs], axis=1)


def apply_multi_slab(src_bits, weights, coeffs, bases, n_covs, s, inv_freq, is_key, pairing=ROPE_HALF):
    """Eq. 8 applied to one (layer, head) slab: C_hat[t] = Align_s(src[t]) + sum_v w_v[t] c_v[t] . B_v,
    anchor v contributing on its covered rows t < n_cov_v.  weights [V, T] (None: all ones).
    Returns (ref, out_bits) like apply_slab; rows no anchor covers keep the aligned source."""
    x = bf16_to_f64(src_bits)
    T = x.shape[0]
    shift = s if is_key else 0
    aligned = rope_shift(x, shift, inv_freq, pairing)
    ref = np.array(aligned, dtype=np.float64, copy=True)
    top = 0
    for v, (c, b, n) in enumerate(zip(coeffs, bases, n_covs)):
        n = min(int(n), T)
        if n <= 0 or np.asarray(b).shape[0] == 0:
            continue
        w = np.ones(n) if weights is None else np.asarray(weights[v], np.float64)[:n]
        ref[:n] += w[:, None] * (np.asarray(c[:n], np.float64) @ np.asarray(b, np.float64))
        top = max(top, n)
    out = f64_to_bf16_bits(ref)
    if shift == 0:
        out[top:] = src_bits[top:]
    return ref, out


# --------------------------------------------------------------------------
# bookkeeping pinned by the paper's memory example (Sec. 3.1)
# --------------------------------------------------------------------------


def full_state_bytes(n_anchors, n_agents, tokens, layers, kv_heads, head_dim, bytes_per_el=2):
    """Full-dimensional anchor pool: each anchor keeps 1 base cache + n_agents deltas,
    keys and values, every layer: O(V N L D)."""
    per_token = 2 * layers * kv_heads * head_dim * bytes_per_el
    return n_anchors * (1 + n_agents) * tokens * per_token


def lowrank_state_bytes(n_anchors, n_agents, tokens, layers, kv_heads, head_dim, r,
                        coeff_bytes=4, basis_bytes=4):
    """Low-rank pool with one state per (layer, KV head): O(V N r (L + D))."""
    per_state = 2 * layers * kv_heads * (tokens * r * coeff_bytes + r * head_dim * basis_bytes)
    return n_anchors * (1 + n_agents) * per_state
