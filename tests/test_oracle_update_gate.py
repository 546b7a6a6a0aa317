"""Pins for the oracle's state update (Eqs. 7, 12), the multi-anchor estimate and
gate (Eqs. 8-11) and the state-size bookkeeping (Sec. 3.1 memory example).

The factorisation is checked against library SVDs (numpy / torch, fp64), the
Eckart-Young optimum and closed-form eigenproblems -- none of which is the
oracle's own Jacobi routine.
"""
import math
import os

import numpy as np
import torch

from oracle import kvc_oracle as orc


def _bits(x):
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def _val(bits):
    return torch.from_numpy(np.asarray(bits).view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()


def test_jacobi_closed_forms():
    # 2x2: [[2,1],[1,2]] has eigenvalues 1 and 3 with eigenvectors (1,-1)/sqrt2, (1,1)/sqrt2
    w, V = orc.jacobi_eigh(np.array([[2.0, 1.0], [1.0, 2.0]]))
    order = np.argsort(w)
    assert np.allclose(w[order], [1.0, 3.0], atol=1e-14)
    assert np.allclose(np.abs(V[:, order[1]]), [1 / math.sqrt(2)] * 2, atol=1e-14)
    # second-difference matrix tridiag(-1, 2, -1) of order n: eigenvalues 2 - 2 cos(k pi/(n+1))
    n = 12
    A = 2 * np.eye(n) - np.eye(n, k=1) - np.eye(n, k=-1)
    w, V = orc.jacobi_eigh(A)
    exp = 2 - 2 * np.cos(np.arange(1, n + 1) * math.pi / (n + 1))
    assert np.allclose(np.sort(w), np.sort(exp), atol=1e-13)
    assert np.allclose(V.T @ V, np.eye(n), atol=1e-13)
    assert np.allclose(A @ V, V * w, atol=1e-12)


def test_fit_matches_library_svd_and_eckart_young():
    rng = np.random.default_rng(0)
    T, d, r = 90, 24, 6
    delta = rng.standard_normal((T, d)) @ np.diag(np.linspace(3.0, 0.1, d)) @ rng.standard_normal((d, d))
    B, w = orc.fit_basis(delta, r)
    A = orc.project(delta, B)
    U, S, Vt = np.linalg.svd(delta, full_matrices=False)
    S_t = torch.linalg.svdvals(torch.from_numpy(delta)).numpy()
    # eigenvalues of the Gram matrix are the squared singular values, sorted descending
    assert np.allclose(w, S ** 2, rtol=1e-10)
    assert np.allclose(w, S_t ** 2, rtol=1e-10)
    # B rows orthonormal, equal to the top right singular vectors up to sign
    assert np.allclose(B @ B.T, np.eye(r), atol=1e-12)
    assert np.allclose(np.abs(np.sum(B * Vt[:r], axis=1)), 1.0, atol=1e-9)
    # sign convention: the largest-magnitude entry of each row is positive
    assert np.all(B[np.arange(r), np.argmax(np.abs(B), axis=1)] > 0)
    # A = U_r Sigma_r: columns orthogonal with norms sigma_1 >= ... >= sigma_r
    Gm = A.T @ A
    assert np.allclose(Gm, np.diag(S[:r] ** 2), atol=1e-8 * S[0] ** 2)
    assert np.allclose(np.abs(A), np.abs(U[:, :r] * S[:r]), atol=1e-8 * S[0])
    # Eckart-Young: the residual is the tail energy
    res = np.sum((delta - A @ B) ** 2)
    assert math.isclose(res, np.sum(S[r:] ** 2), rel_tol=1e-9)
    # and no other rank-r projection does better (random subspaces)
    for _ in range(5):
        Q = np.linalg.qr(rng.standard_normal((d, r)))[0].T
        assert np.sum((delta - (delta @ Q.T) @ Q) ** 2) >= res * (1 - 1e-12)


def test_exact_rank_r_deviation_is_reconstructed_to_rounding():
    # a deviation built exactly rank r (coeff x orthonormal basis) comes back to fp64 rounding
    rng = np.random.default_rng(1)
    T, d, r = 256, 64, 8
    c = rng.standard_normal((T, r))
    Bt = np.linalg.qr(rng.standard_normal((d, r)))[0].T
    delta = c @ Bt
    B, w = orc.fit_basis(delta, r)
    A = orc.project(delta, B)
    assert np.max(np.abs(A @ B - delta)) < 1e-12
    assert np.all(np.abs(w[r:]) < 1e-12 * w[0])
    # same subspace as the construction
    assert np.allclose(B.T @ B, Bt.T @ Bt, atol=1e-10)
    # full rank r = d reconstructs anything
    delta = rng.standard_normal((40, 16))
    B, _ = orc.fit_basis(delta, 16)
    assert np.max(np.abs(orc.project(delta, B) @ B - delta)) < 1e-12


def test_rank_limits_and_selection_basis():
    rng = np.random.default_rng(2)
    # fewer rows than the requested rank: rows beyond T are zero
    delta = rng.standard_normal((3, 8))
    B, w = orc.fit_basis(delta, 5)
    assert np.allclose(B[3:], 0) and np.allclose(B[:3] @ B[:3].T, np.eye(3), atol=1e-12)
    # projecting on unit rows picks channels
    delta = rng.standard_normal((7, 8))
    sel = np.eye(8)[[5, 0, 2]]
    assert np.array_equal(orc.project(delta, sel), delta[:, [5, 0, 2]])


def test_state_update_then_apply_round_trip():
    # target = Align(src) + exact rank-r deviation (kept in float64, not re-quantised):
    # FIT then the unrounded apply reproduces it to rounding; the first hop of a chain.
    rng = np.random.default_rng(3)
    L, H, T, d, r, s = 1, 2, 48, 16, 4, 16
    f = orc.rope_inv_freq(d, 10000.0)
    src = orc.Cache(_bits(rng.standard_normal((L, H, T, d))), _bits(rng.standard_normal((L, H, T, d))))
    for l in range(L):
        for h in range(H):
            c = rng.standard_normal((T, r))
            Bt = np.linalg.qr(rng.standard_normal((d, r)))[0].T
            aligned = orc.rope_shift(_val(src.k[l, h]), s, f)
            target = aligned + c @ Bt
            dlt = target - aligned
            B, _ = orc.fit_basis(dlt, r)
            out = orc.chain_unrounded_slab(_val(src.k[l, h]), [0, s], [orc.project(dlt, B)], [B], f, True)[0]
            assert np.max(np.abs(out - target)) < 1e-12


def test_state_update_deviation_uses_aligned_source():
    # Eq. 12: Delta = C_j - Align(C_i).  If the target is exactly the re-aligned source the
    # key deviation vanishes; values ignore the shift.
    rng = np.random.default_rng(4)
    d, T, s = 8, 5, 11
    f = orc.rope_inv_freq(d, 10000.0)
    src = _bits(rng.standard_normal((T, d)))
    aligned = orc.rope_shift(_val(src), s, f)
    dk = orc.deviation(src, src, s, f, is_key=True)
    assert np.allclose(dk, _val(src) - aligned, atol=1e-15) and np.max(np.abs(dk)) > 0.1
    assert np.array_equal(orc.deviation(src, src, s, f, is_key=False), np.zeros((T, d)))
    # src None: factorise the cache itself
    assert np.array_equal(orc.deviation(None, src, s, f, is_key=True), _val(src))


def test_state_update_project_mode_full():
    rng = np.random.default_rng(5)
    L, H, T, d, r, s = 2, 1, 12, 8, 3, -4
    f = orc.rope_inv_freq(d, 10000.0)
    src = orc.Cache(_bits(rng.standard_normal((L, H, T, d))), _bits(rng.standard_normal((L, H, T, d))))
    tgt = orc.Cache(_bits(rng.standard_normal((L, H, T, d))), _bits(rng.standard_normal((L, H, T, d))))
    bk = rng.standard_normal((L, H, r, d)).astype(np.float32)
    bv = rng.standard_normal((L, H, r, d)).astype(np.float32)
    st, _ = orc.state_update(src, tgt, s, f, mode=orc.PROJECT, basis_k=bk, basis_v=bv)
    assert st.coeff_k.dtype == np.float32 and st.coeff_k.shape == (L, H, T, r)
    # scalar re-derivation of a few entries
    for (l, t, q) in ((0, 0, 0), (1, 7, 2), (1, 11, 1)):
        acc_k = acc_v = 0.0
        ks, kt = _val(src.k[l, 0, t]), _val(tgt.k[l, 0, t])
        for c in range(d):
            k = c % (d // 2)
            ang = s * 10000.0 ** (-2.0 * k / d)
            rot = (ks[k] * math.cos(ang) - ks[k + d // 2] * math.sin(ang)) if c < d // 2 else \
                  (ks[k] * math.sin(ang) + ks[k + d // 2] * math.cos(ang))
            acc_k += (kt[c] - rot) * float(bk[l, 0, q, c])
            acc_v += (_val(tgt.v[l, 0, t])[c] - _val(src.v[l, 0, t])[c]) * float(bv[l, 0, q, c])
        assert math.isclose(float(st.coeff_k[l, 0, t, q]), acc_k, rel_tol=1e-6, abs_tol=1e-6)
        assert math.isclose(float(st.coeff_v[l, 0, t, q]), acc_v, rel_tol=1e-6, abs_tol=1e-6)


# ---- gate and multi-anchor estimate (Eqs. 8-11) -----------------------------


def test_entropy_limits():
    for n in (2, 5, 10):
        assert math.isclose(orc.normalized_entropy(np.full(n, 1.0 / n)), 1.0, rel_tol=1e-12)
        one_hot = np.zeros(n)
        one_hot[1] = 1.0
        assert orc.normalized_entropy(one_hot) == 0.0
    # two anchors, weights (1/4, 3/4): H = 2 - (3/4) log2 3
    assert math.isclose(orc.normalized_entropy(np.array([0.25, 0.75])), 2 - 0.75 * math.log2(3), rel_tol=1e-12)
    try:
        orc.normalized_entropy(np.array([1.0]))
        assert False, "a single anchor has no gate value"
    except ValueError:
        pass


def test_gate_weights_and_distance():
    g = orc.gate_weights(np.array([1.0, 1.0, 1.0]))
    assert np.allclose(g, 1 / 3)
    g = orc.gate_weights(np.array([0.0, math.log(3.0)]))        # exp(0) : exp(-ln 3) = 3 : 1
    assert np.allclose(g, [0.75, 0.25])
    # distance: two layers, prefix k = 2; differences 3 and 4 in single entries -> 5
    a = [np.zeros((3, 2)), np.zeros((3, 2))]
    b = [np.array([[3.0, 0], [0, 0], [9, 9]]), np.array([[0, 0], [0, 4.0], [9, 9]])]
    assert math.isclose(orc.gate_distance(a, b, 2), 5.0)


def test_multi_anchor_is_apply_at_stacked_rank():
    rng = np.random.default_rng(6)
    V, T, r, d = 3, 10, 4, 8
    w = rng.random((V, T))
    w /= w.sum(0, keepdims=True)
    As = [rng.standard_normal((T, r)) for _ in range(V)]
    Bs = [rng.standard_normal((r, d)) for _ in range(V)]
    est = orc.multi_anchor_delta(w, As, Bs)
    # scalar definition of Eq. 8 for one entry
    t, c = 4, 5
    ref = sum(w[v, t] * sum(As[v][t, q] * Bs[v][q, c] for q in range(r)) for v in range(V))
    assert math.isclose(est[t, c], ref, rel_tol=1e-12)
    cs, bs = orc.stack_anchors(w, As, Bs)
    assert cs.shape == (T, V * r) and bs.shape == (V * r, d)
    assert np.allclose(cs @ bs, est, atol=1e-12)
    # a single anchor with weight one is the plain correction
    assert np.allclose(orc.multi_anchor_delta(np.ones((1, T)), As[:1], Bs[:1]), As[0] @ Bs[0])


# ---- bookkeeping --------------------------------------------------------------


def test_memory_example_from_the_paper():
    path = os.path.join(os.path.dirname(__file__), "golden", "memory_example.txt")
    row = [ln for ln in open(path) if ln.strip() and not ln.startswith("#")][0].split()
    L, Hkv, hd, bpe, tok, V, N = (int(x) for x in row[:7])
    expect, tol = float(row[7]), float(row[8])
    got = orc.full_state_bytes(V, N, tok, L, Hkv, hd, bpe) / 2.0 ** 30
    assert abs(got - expect) <= tol
    # the low-rank pool is O(V N r (L_seg + D)) per matrix
    lr = orc.lowrank_state_bytes(V, N, tok, L, Hkv, hd, r=32)
    per_matrix = 32 * (tok + hd) * 4
    assert lr == V * (1 + N) * 2 * L * Hkv * per_matrix
    # counted, not computed: allocate a tiny pool's factors (a base factorisation and N corrections per
    # anchor, keys and values, one state per (layer, KV head)) and add up what the arrays occupy
    v, n, t, l, h, d, r = 3, 2, 7, 2, 3, 8, 4
    arrays = []
    for _anchor in range(v):
        for _state in range(1 + n):
            for _kv in range(2):
                arrays.append(np.zeros((l, h, t, r), np.float32))       # coefficients
                arrays.append(np.zeros((l, h, r, d), np.float32))       # basis
    assert orc.lowrank_state_bytes(v, n, t, l, h, d, r) == sum(a.nbytes for a in arrays)
    full = [np.zeros((l, h, t, d), np.float16) for _ in range(v * (1 + n) * 2)]   # 2-byte elements, like bf16
    assert orc.full_state_bytes(v, n, t, l, h, d, 2) == sum(a.nbytes for a in full)
    # the scaling the paper states: for long segments the ratio full / low-rank tends to D b_full / (r b_coeff)
    big = 1 << 22
    ratio = orc.full_state_bytes(1, 1, big, 1, 1, 128, 2) / orc.lowrank_state_bytes(1, 1, big, 1, 1, 128, 32)
    assert abs(ratio - 128 * 2 / (32 * 4)) < 1e-3


def test_token_weights_pins():
    rng = np.random.default_rng(3)
    T, F = 7, 12
    x = rng.standard_normal((T, F))
    # identical anchors: uniform weights; a single anchor: all ones
    a = rng.standard_normal((T, F))
    w = orc.token_weights(x, [a, a, a])
    assert np.allclose(w, 1.0 / 3.0)
    assert np.allclose(orc.token_weights(x, [a]), 1.0)
    # columns sum to one; hand-computed two-anchor case: scores m0, m1 -> w0 = 1 / (1 + exp(m0 - m1))
    b = rng.standard_normal((T, F))
    w = orc.token_weights(x, [a, b])
    assert np.allclose(w.sum(axis=0), 1.0)
    m0 = np.abs(x - a).mean(axis=1)
    m1 = np.abs(x - b).mean(axis=1)
    assert np.allclose(w[0], 1.0 / (1.0 + np.exp(m0 - m1)))
    # the anchor that equals the source on a token gets the larger weight there, and almost all of it
    # when the other is far away
    far = x + 100.0
    near = x.copy()
    w = orc.token_weights(x, [near, far])
    assert np.all(w[0] > 1.0 - 1e-12)
    # token-wise: swapping which anchor is near on the second half swaps the weights there
    mix = np.where(np.arange(T)[:, None] < 3, near, far)
    mix2 = np.where(np.arange(T)[:, None] < 3, far, near)
    w = orc.token_weights(x, [mix, mix2])
    assert np.all(w[0, :3] > 0.999) and np.all(w[1, 3:] > 0.999)
    # a temperature rescales the scores: T -> infinity gives uniform weights
    assert np.allclose(orc.token_weights(x, [a, b], temperature=1e12), 0.5, atol=1e-9)


def test_apply_multi_slab_pins():
    rng = np.random.default_rng(4)
    T, d, r = 9, 8, 3
    inv = orc.rope_inv_freq(d, 10000.0)
    src = orc.f64_to_bf16_bits(rng.standard_normal((T, d)))
    cs = [rng.standard_normal((T, r)) for _ in range(3)]
    bs = [rng.standard_normal((r, d)) for _ in range(3)]
    w = rng.random((3, T))
    w /= w.sum(axis=0, keepdims=True)
    for is_key, s in ((True, 5), (False, 5), (True, 0)):
        ref, out = orc.apply_multi_slab(src, w, cs, bs, [T, T, T], s, inv, is_key)
        # equals the single-state apply at the stacked rank (weights folded into the coefficients)
        c_st, b_st = orc.stack_anchors(w, cs, bs)
        ref1, out1 = orc.apply_slab(src, c_st, b_st, s, inv, T, is_key)
        assert np.allclose(ref, ref1, rtol=0, atol=1e-12) and np.array_equal(out, out1)
        # and the aligned source plus Eq. 8's estimate
        base = orc.rope_shift(orc.bf16_to_f64(src), s if is_key else 0, inv)
        assert np.allclose(ref, base + orc.multi_anchor_delta(w, cs, bs), atol=1e-12)
    # one anchor, unit weights: the plain apply
    ref, out = orc.apply_multi_slab(src, None, cs[:1], bs[:1], [T], 3, inv, True)
    ref1, out1 = orc.apply_slab(src, cs[0], bs[0], 3, inv, T, True)
    assert np.array_equal(ref, ref1) and np.array_equal(out, out1)
    # partial coverage per anchor: rows beyond an anchor's length get nothing from it; rows beyond
    # every anchor keep the source bits at shift 0
    ref, out = orc.apply_multi_slab(src, w, cs, bs, [4, 6, 0], 0, inv, False)
    x = orc.bf16_to_f64(src)
    exp = x.copy()
    exp[:4] += w[0, :4, None] * (cs[0][:4] @ bs[0])
    exp[:6] += w[1, :6, None] * (cs[1][:6] @ bs[1])
    assert np.allclose(ref, exp, atol=1e-12) and np.array_equal(out[6:], src[6:])
    # canonical key features: rotating a cache forward by p and asking for canonical coordinates undoes it
    k = rng.standard_normal((T, d))
    moved = orc.rope_shift(k, 11, inv)
    assert np.allclose(orc.canonical_key_features([moved], 11, inv), k, atol=1e-12)


def test_realign_basis_pins():
    """Rot_s(c . B) = c . Rot_s(B); canonical storage: a correction fitted at target position p and
    re-aligned by -p equals the correction fitted on inputs that were first moved to position 0."""
    rng = np.random.default_rng(6)
    T, d, r = 11, 8, 3
    inv = orc.rope_inv_freq(d, 10000.0)
    c = rng.standard_normal((T, r))
    B = rng.standard_normal((r, d))
    for s in (0, 7, -19):
        lhs = orc.rope_shift(c @ B, s, inv)
        assert np.allclose(lhs, c @ orc.realign_basis(B, s, inv), atol=1e-12)
    assert np.array_equal(orc.realign_basis(B, 0, inv), B)
    assert np.allclose(orc.realign_basis(orc.realign_basis(B, 5, inv), -5, inv), B, atol=1e-12)
    # rows stay orthonormal (a rotation is orthogonal)
    Q = np.linalg.qr(rng.standard_normal((d, r)))[0].T
    Qr = orc.realign_basis(Q, 13, inv)
    assert np.allclose(Qr @ Qr.T, np.eye(r), atol=1e-12)
    # the deviation measured at target position p_t, moved back to position 0, is the deviation of the
    # inputs moved back to their canonical coordinates: coefficients on the re-aligned basis agree
    p_s, p_t = 40, 95
    src = rng.standard_normal((T, d))
    tgt = orc.rope_shift(src, p_t - p_s, inv) + c @ Q
    delta_t = tgt - orc.rope_shift(src, p_t - p_s, inv)                       # Eq. 12, at the target's positions
    delta_0 = orc.rope_shift(tgt, -p_t, inv) - orc.rope_shift(src, -p_s, inv)  # both sides canonical
    assert np.allclose(orc.rope_shift(delta_t, -p_t, inv), delta_0, atol=1e-12)
    assert np.allclose(delta_t @ Q.T, delta_0 @ orc.realign_basis(Q, -p_t, inv).T, atol=1e-12)


def test_effective_rank_pins():
    # one dominant direction: rank 1 keeps it all
    assert orc.effective_rank([10.0, 0.0, 0.0]) == 1
    # k equal eigenvalues: 90 % of the energy needs ceil(0.9 k) of them
    for k in (1, 2, 5, 10, 32):
        assert orc.effective_rank(np.ones(k)) == math.ceil(0.9 * k - 1e-12)
    # hand case: energies 50, 30, 15, 5 -> cumulative 50, 80, 95: three directions reach 90 %
    assert orc.effective_rank([5.0, 50.0, 15.0, 30.0]) == 3
    assert orc.effective_rank([50.0, 30.0, 10.0, 10.0]) == 3          # exactly 90 % after three
    assert orc.effective_rank([50.0, 30.0, 15.0, 5.0], energy=0.8) == 2
    assert orc.effective_rank([0.0, 0.0]) == 0 and orc.effective_rank([-1e-9, 0.0]) == 0
    # the singular values of a matrix: energy = squared singular values (library SVD)
    rng = np.random.default_rng(9)
    m = rng.standard_normal((40, 6)) @ np.diag([9.0, 5.0, 2.0, 1.0, 0.5, 0.1]) @ rng.standard_normal((6, 12))
    sv = np.linalg.svd(m, compute_uv=False)
    e = sv ** 2
    k = orc.effective_rank(np.linalg.eigvalsh(m.T @ m))
    assert e[:k].sum() >= 0.9 * e.sum() > e[:k - 1].sum()


def test_grouped_state_pins():
    """D = H d: the grouped state is the plain low-rank product on the concatenated feature axis."""
    rng = np.random.default_rng(8)
    L, H, T, d, r = 2, 3, 5, 4, 2
    ck, cv = rng.standard_normal((L, T, r)), rng.standard_normal((L, T, r))
    bk, bv = rng.standard_normal((L, r, H * d)), rng.standard_normal((L, r, H * d))
    st = orc.ungroup_state(ck, cv, bk, bv, H)
    assert st.coeff_k.shape == (L, H, T, r) and st.basis_k.shape == (L, H, r, d)
    for l in range(L):
        z = cv[l] @ bv[l]                                             # [T, H d]
        per_head = np.concatenate([st.coeff_v[l, h] @ st.basis_v[l, h] for h in range(H)], axis=1)
        assert np.allclose(z, per_head, atol=1e-12)
    # the projection of a concatenated deviation is the sum of the heads' projections
    delta = [rng.standard_normal((T, d)) for _ in range(H)]
    c = orc.project_grouped(delta, bk[0])
    by_head = sum(orc.project(delta[h], st.basis_k[0, h]) for h in range(H))
    assert np.allclose(c, by_head, atol=1e-12)
    # orthonormal rows in R^{H d}: projecting c @ B gives c back
    Q = np.linalg.qr(rng.standard_normal((H * d, r)))[0].T
    z = ck[0] @ Q
    assert np.allclose(orc.project_grouped([z[:, h * d:(h + 1) * d] for h in range(H)], Q), ck[0], atol=1e-12)
    # compactness (Sec. 3.1): float32 coefficients of a grouped state take r*4 / (H*d*2) of the bf16 cache
    assert math.isclose((r * 4) / (H * d * 2), 8 / 24)


def test_grouped_fit_matches_library_svd():
    """D = H d fit (Sec. 3.1, Eq. 7): the oracle's grouped basis spans the library SVD's leading right
    singular subspace of the concatenated deviation, its eigenvalues are the squared singular values,
    and a deviation built exactly rank r across the heads is reconstructed to rounding.  A per-head
    fit of the same data does NOT reproduce it (the heads share coefficients only under grouping)."""
    rng = np.random.default_rng(21)
    H, T, d, r = 3, 40, 6, 4
    c = rng.standard_normal((T, r))
    Q = np.linalg.qr(rng.standard_normal((H * d, r)))[0].T                 # orthonormal rows in R^{H d}
    cat = c @ Q + 1e-4 * rng.standard_normal((T, H * d))
    slabs = [cat[:, h * d:(h + 1) * d] for h in range(H)]
    B, w = orc.fit_grouped(slabs, r)
    sv = np.linalg.svd(cat, compute_uv=False)
    assert np.allclose(w[:H * d], sv[:H * d] ** 2 if sv.size >= H * d else np.concatenate([sv ** 2, np.zeros(H * d - sv.size)]),
                       rtol=1e-9, atol=1e-12)
    Vt = np.linalg.svd(cat, full_matrices=False)[2][:r]
    assert np.linalg.norm(B.T @ B - Vt.T @ Vt) <= 1e-8
    assert np.allclose(B @ B.T, np.eye(r), atol=1e-12)
    # exactly rank r: reconstructed to rounding, with coefficients shared by the heads
    exact = c @ Q
    Be, _ = orc.fit_grouped([exact[:, h * d:(h + 1) * d] for h in range(H)], r)
    ce = orc.project_grouped([exact[:, h * d:(h + 1) * d] for h in range(H)], Be)
    assert np.max(np.abs(ce @ Be - exact)) <= 1e-12
    # per-head rank-r fits of the same data need H sets of coefficients to do the same
    per_head = [orc.fit_basis(exact[:, h * d:(h + 1) * d], r)[0] for h in range(H)]
    assert all(np.max(np.abs(orc.project(exact[:, h * d:(h + 1) * d], per_head[h]) @ per_head[h]
                             - exact[:, h * d:(h + 1) * d])) <= 1e-12 for h in range(H))
    assert not np.allclose(orc.project(exact[:, :d], per_head[0]), ce)


def test_state_update_fit_wrapper_against_library_svd():
    """state_update(FIT) as a whole (the covered prefix, the float32 storage of the basis that then
    projects, keys against the aligned source, values unshifted) against a library SVD of deviations
    re-derived here with scalar rotations: the coefficient Gram matrix carries the squared singular
    values, coeff . basis is the best rank-r approximation of the covered rows, rows beyond n_cov do not
    influence anything."""
    rng = np.random.default_rng(77)
    L, H, T, d, r, n_cov, s = 1, 2, 19, 8, 3, 13, 5
    f = orc.rope_inv_freq(d, 10000.0)
    sk, sv = _bits(rng.standard_normal((L, H, T, d))), _bits(rng.standard_normal((L, H, T, d)))
    tk, tv = _bits(rng.standard_normal((L, H, T, d))), _bits(rng.standard_normal((L, H, T, d)))
    src, tgt = orc.Cache(sk, sv), orc.Cache(tk, tv)
    st, ev = orc.state_update(src, tgt, s, f, r=r, mode=orc.FIT, n_cov=n_cov)
    assert st.coeff_k.shape == (L, H, n_cov, r) and st.coeff_k.dtype == np.float32 and st.basis_k.dtype == np.float32
    # changing the uncovered rows changes nothing
    tk2 = tk.copy()
    tk2[:, :, n_cov:] = _bits(rng.standard_normal((L, H, T - n_cov, d)))
    st2, ev2 = orc.state_update(src, orc.Cache(tk2, tv), s, f, r=r, mode=orc.FIT, n_cov=n_cov)
    assert np.array_equal(st2.basis_k, st.basis_k) and np.array_equal(st2.coeff_k, st.coeff_k) and np.array_equal(ev2, ev)
    for h in range(H):
        # keys: tgt - Rot_s(src), the rotation written out per pair with math functions
        x, y = _val(sk[0, h]), _val(tk[0, h])
        dk = np.zeros((n_cov, d))
        for t in range(n_cov):
            for k in range(d // 2):
                c, sn = math.cos(s * f[k]), math.sin(s * f[k])
                dk[t, k] = y[t, k] - (x[t, k] * c - x[t, k + d // 2] * sn)
                dk[t, k + d // 2] = y[t, k + d // 2] - (x[t, k] * sn + x[t, k + d // 2] * c)
        dv = (_val(tv[0, h]) - _val(sv[0, h]))[:n_cov]
        for dl, B, c, w in ((dk, st.basis_k[0, h], st.coeff_k[0, h], ev[0, h, 0]), (dv, st.basis_v[0, h], st.coeff_v[0, h], ev[0, h, 1])):
            U, S, Vt = np.linalg.svd(dl, full_matrices=False)
            assert np.allclose(w[:len(S)], S ** 2, rtol=1e-9, atol=1e-12)
            B64, c64 = B.astype(np.float64), c.astype(np.float64)
            best = (U[:, :r] * S[:r]) @ Vt[:r]
            assert np.max(np.abs(c64 @ B64 - best)) <= 1e-5             # float32 storage of both factors
            assert np.max(np.abs(c64.T @ c64 - np.diag(S[:r] ** 2))) <= 1e-4 * S[0] ** 2
            assert np.allclose(c64, dl @ B64.T, atol=1e-6)               # the STORED (float32) basis is what projects
