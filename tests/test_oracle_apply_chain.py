"""Pins for the oracle's apply / chain / paged addressing.

Brute force on tiny inputs is written here with scalar Python loops and
``math`` only, from the definitions (Eq. 8 with one anchor, the chained
recursion of Sec. 3.2), not by calling back into the oracle.
"""
import math

import numpy as np
import torch

from oracle import kvc_oracle as orc


def _bits(x):
    """float -> bf16 bits through torch (independent of the oracle's codec)."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def _val(bits):
    return torch.from_numpy(np.asarray(bits).view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()


def _rand_cache(rng, L, H, T, d):
    return orc.Cache(_bits(rng.standard_normal((L, H, T, d))), _bits(rng.standard_normal((L, H, T, d))))


def _rand_state(rng, L, H, T, d, r, n_cov=None):
    n = T if n_cov is None else n_cov
    q = np.linalg.qr(rng.standard_normal((L, H, d, r)))[0].transpose(0, 1, 3, 2)
    q2 = np.linalg.qr(rng.standard_normal((L, H, d, r)))[0].transpose(0, 1, 3, 2)
    return orc.State(rng.standard_normal((L, H, n, r)).astype(np.float32),
                     rng.standard_normal((L, H, n, r)).astype(np.float32),
                     q.astype(np.float32), q2.astype(np.float32), n_cov=n)


def _brute_apply(src, st, s, theta, n_cov):
    """Element-by-element definition: returns float64 [2][L][H][T][d] before rounding."""
    L, H, T, d = src.L, src.H, src.T, src.d
    out = np.zeros((2, L, H, T, d))
    kv = (_val(src.k), _val(src.v))
    for l in range(L):
        for h in range(H):
            for t in range(T):
                for c in range(d):
                    # keys: rotate the pair (c mod d/2, c mod d/2 + d/2) by s * theta^(-2k/d)
                    k = c % (d // 2)
                    ang = s * theta ** (-2.0 * k / d)
                    x1, x2 = kv[0][l, h, t, k], kv[0][l, h, t, k + d // 2]
                    if c < d // 2:
                        a = x1 * math.cos(ang) - x2 * math.sin(ang)
                    else:
                        a = x1 * math.sin(ang) + x2 * math.cos(ang)
                    vv = kv[1][l, h, t, c]
                    if t < n_cov:
                        for q in range(st.r):
                            a += float(st.coeff_k[l, h, t, q]) * float(st.basis_k[l, h, q, c])
                            vv += float(st.coeff_v[l, h, t, q]) * float(st.basis_v[l, h, q, c])
                    out[0, l, h, t, c] = a
                    out[1, l, h, t, c] = vv
    return out


def test_apply_matches_brute_force_tiny():
    rng = np.random.default_rng(0)
    L, H, T, d, r, theta, s, n_cov = 2, 2, 7, 8, 3, 10000.0, 5, 5
    src = _rand_cache(rng, L, H, T, d)
    st = _rand_state(rng, L, H, T, d, r, n_cov)
    dst, rk, rv = orc.apply(src, st, s, orc.rope_inv_freq(d, theta), want_ref=True)
    brute = _brute_apply(src, st, s, theta, n_cov)
    assert np.allclose(rk, brute[0], atol=1e-13)
    assert np.allclose(rv, brute[1], atol=1e-13)
    # materialised cache = the brute-force value rounded once by torch
    assert np.array_equal(dst.k, _bits(brute[0]))
    assert np.array_equal(dst.v, _bits(brute[1]))
    # values never rotate: rows beyond the covered prefix are the source bits
    assert np.array_equal(dst.v[:, :, n_cov:], src.v[:, :, n_cov:])
    # keys beyond the covered prefix are rotated only
    assert not np.array_equal(dst.k[:, :, n_cov:], src.k[:, :, n_cov:])


def test_empty_state_is_bit_identity():
    rng = np.random.default_rng(1)
    L, H, T, d = 1, 2, 9, 16
    src = _rand_cache(rng, L, H, T, d)
    # exotic patterns must survive: -0.0, inf, NaN payload, subnormal
    src.k[0, 0, 0, :4] = [0x8000, 0x7F80, 0x7FC1, 0x0001]
    src.v[0, 1, 3, :4] = [0x8000, 0xFF80, 0xFFC5, 0x8001]
    f = orc.rope_inv_freq(d, 10000.0)
    empty = orc.State(np.zeros((L, H, 0, 0), np.float32), np.zeros((L, H, 0, 0), np.float32),
                      np.zeros((L, H, 0, d), np.float32), np.zeros((L, H, 0, d), np.float32), n_cov=0)
    out = orc.apply(src, empty, 0, f)
    assert np.array_equal(out.k, src.k) and np.array_equal(out.v, src.v)
    # rank > 0 but nothing covered: same
    st = _rand_state(rng, L, H, T, d, 4, n_cov=0)
    out = orc.apply(src, st, 0, f)
    assert np.array_equal(out.k, src.k) and np.array_equal(out.v, src.v)
    # with a shift the values are still bit-identical, the keys are rotated
    out = orc.apply(src, empty, 3, f)
    assert np.array_equal(out.v, src.v)
    assert not np.array_equal(out.k, src.k)


def test_zero_coefficients_leave_finite_values_unchanged():
    rng = np.random.default_rng(2)
    L, H, T, d, r = 1, 1, 6, 8, 2
    src = _rand_cache(rng, L, H, T, d)
    st = _rand_state(rng, L, H, T, d, r)
    st.coeff_k[:] = 0
    st.coeff_v[:] = 0
    out = orc.apply(src, st, 0, orc.rope_inv_freq(d, 10000.0))
    assert np.array_equal(_val(out.k), _val(src.k)) and np.array_equal(_val(out.v), _val(src.v))


def test_apply_is_linear_in_the_state():
    # stacking two rank-r states as one rank-2r state adds their corrections
    rng = np.random.default_rng(3)
    L, H, T, d, r = 1, 2, 11, 16, 3
    src = _rand_cache(rng, L, H, T, d)
    a, b = _rand_state(rng, L, H, T, d, r), _rand_state(rng, L, H, T, d, r)
    both = orc.State(np.concatenate([a.coeff_k, b.coeff_k], -1), np.concatenate([a.coeff_v, b.coeff_v], -1),
                     np.concatenate([a.basis_k, b.basis_k], 2), np.concatenate([a.basis_v, b.basis_v], 2))
    f = orc.rope_inv_freq(d, 10000.0)
    s = 9
    _, ka, va = orc.apply(src, a, s, f, want_ref=True)
    _, kb, vb = orc.apply(src, b, s, f, want_ref=True)
    _, k2, v2 = orc.apply(src, both, s, f, want_ref=True)
    base_k = orc.rope_shift(_val(src.k), s, f)
    assert np.allclose(k2 - base_k, (ka - base_k) + (kb - base_k), atol=1e-12)
    assert np.allclose(v2 - _val(src.v), (va - _val(src.v)) + (vb - _val(src.v)), atol=1e-12)


def test_chain_first_agent_untouched_and_matches_stepwise_brute_force():
    rng = np.random.default_rng(4)
    L, H, T, d, r, theta = 1, 2, 5, 8, 2, 10000.0
    prefix = [32, 48, 40, 71]
    a0 = _rand_cache(rng, L, H, T, d)
    k0, v0 = a0.k.copy(), a0.v.copy()
    states = [_rand_state(rng, L, H, T, d, r) for _ in range(3)]
    outs = orc.chain(a0, prefix, states, orc.rope_inv_freq(d, theta))
    assert np.array_equal(a0.k, k0) and np.array_equal(a0.v, v0)
    assert len(outs) == 3
    # brute force, hop by hop, rounding to bf16 at every hop with torch
    cur = orc.Cache(k0.copy(), v0.copy())
    for a in range(1, 4):
        brute = _brute_apply(cur, states[a - 1], prefix[a] - prefix[a - 1], theta, T)
        cur = orc.Cache(_bits(brute[0]), _bits(brute[1]))
        assert np.array_equal(outs[a - 1].k, cur.k)
        assert np.array_equal(outs[a - 1].v, cur.v)


def test_chain_closed_form_by_linearity():
    # without intermediate rounding:
    #   K_a[t] = Rot_{P_a - P_0} K_0[t] + sum_{b<=a} Rot_{P_a - P_b}(c_b[t] B_b)
    rng = np.random.default_rng(5)
    T, d, r, theta = 6, 16, 3, 500000.0
    prefix = [100, 37, 260, 300, 64]
    f = orc.rope_inv_freq(d, theta)
    x0 = rng.standard_normal((T, d))
    cs = [rng.standard_normal((T, r)) for _ in range(4)]
    bs = [rng.standard_normal((r, d)) for _ in range(4)]
    outs = orc.chain_unrounded_slab(x0, prefix, cs, bs, f, is_key=True)
    for a in range(1, 5):
        exp = np.zeros((T, d))
        for t in range(T):
            for k in range(d // 2):
                def rot(vec, s):
                    ang = s * theta ** (-2.0 * k / d)
                    return (vec[k] * math.cos(ang) - vec[k + d // 2] * math.sin(ang),
                            vec[k] * math.sin(ang) + vec[k + d // 2] * math.cos(ang))
                y1, y2 = rot(x0[t], prefix[a] - prefix[0])
                for b in range(1, a + 1):
                    corr = cs[b - 1][t] @ bs[b - 1]
                    z1, z2 = rot(corr, prefix[a] - prefix[b])
                    y1, y2 = y1 + z1, y2 + z2
                exp[t, k], exp[t, k + d // 2] = y1, y2
        assert np.allclose(outs[a - 1], exp, atol=1e-11)
    # values: plain sums
    vouts = orc.chain_unrounded_slab(x0, prefix, cs, bs, f, is_key=False)
    assert np.allclose(vouts[-1], x0 + sum(c @ b for c, b in zip(cs, bs)), atol=1e-12)


def test_chain_rounding_stays_near_unrounded():
    # with bf16 rounding at every hop the result drifts by at most about a * 2^-8 relative
    rng = np.random.default_rng(6)
    L, H, T, d, r = 1, 1, 64, 32, 4
    prefix = [64, 80, 200, 130]
    f = orc.rope_inv_freq(d, 10000.0)
    a0 = _rand_cache(rng, L, H, T, d)
    states = [_rand_state(rng, L, H, T, d, r) for _ in range(3)]
    outs = orc.chain(a0, prefix, states, f)
    un = orc.chain_unrounded_slab(_val(a0.k[0, 0]), prefix, [s.coeff_k[0, 0] for s in states],
                                  [s.basis_k[0, 0] for s in states], f, is_key=True)
    for a in range(3):
        got = _val(outs[a].k[0, 0])
        rownorm = np.linalg.norm(un[a], axis=1, keepdims=True)
        assert np.max(np.abs(got - un[a]) / rownorm) < (a + 1) * 2.0 ** -8


def test_chained_equals_context_free_reference_with_exact_corrections():
    # Eq. 6: Delta_{j<-i} = Delta_{j<-ref} - Delta_{i<-ref}.  With exact (full) corrections,
    # chaining agent to agent reproduces every agent's true cache, exactly as correcting
    # each agent from the reference would.  No positional shift here: the identity is
    # about the reference, not about alignment.
    rng = np.random.default_rng(7)
    T, d = 9, 8
    ref = rng.standard_normal((T, d))
    true = [ref + rng.standard_normal((T, d)) for _ in range(4)]          # C_j
    d_ref = [c - ref for c in true]                                       # Delta_{j<-ref}
    f = orc.rope_inv_freq(d, 10000.0)
    eye = np.eye(d)
    # chained: C_0 exact, hop a uses Delta_{a<-a-1} = d_ref[a] - d_ref[a-1], basis = identity (r = d)
    cs = [d_ref[a] - d_ref[a - 1] for a in range(1, 4)]
    outs = orc.chain_unrounded_slab(true[0], [0, 0, 0, 0], cs, [eye] * 3, f, is_key=True)
    for a in range(1, 4):
        assert np.allclose(outs[a - 1], true[a], atol=1e-13)                      # chained
        assert np.allclose(ref + d_ref[a], true[a], atol=1e-13)                   # non-chained


def test_paged_indexing_bit_exact():
    # injective code of (l, h, t, c) stored as bf16-exact small integers; rank 0, shift 0,
    # two different shuffled page tables: gather and scatter must be exact and unmapped
    # physical pages must keep their sentinel.
    L, H, T, d, page, P = 2, 3, 37, 4, 16, 7          # T is not a multiple of the page size
    npg = (T + page - 1) // page
    rng = np.random.default_rng(8)
    pt_src = rng.permutation(P)[:npg].astype(np.int32)
    pt_dst = rng.permutation(P)[:npg].astype(np.int32)
    code = np.zeros((L, H, T, d), np.uint16)
    for l in range(L):
        for h in range(H):
            for t in range(T):
                for c in range(d):
                    code[l, h, t, c] = 1 + (((l * H + h) * T + t) * d + c)   # < 2^16, distinct, never 0xDEAD
    assert code.max() < 0xDEAD
    pool_k = np.full((L, P, H, page, d), 0xDEAD, np.uint16)
    pool_v = np.full((L, P, H, page, d), 0xDEAD, np.uint16)
    for l in range(L):
        for h in range(H):
            for t in range(T):
                pool_k[l, pt_src[t // page], h, t % page] = code[l, h, t]
                pool_v[l, pt_src[t // page], h, t % page] = code[l, h, t] ^ 0x4000
    src = orc.Cache(pool_k, pool_v, T=T, page_table=pt_src)
    assert np.array_equal(src.get_bits("k", 1, 2), code[1, 2])
    dst = src.empty_like(page_table=pt_dst, fill=0xBEEF)
    empty = orc.State(np.zeros((L, H, 0, 0), np.float32), np.zeros((L, H, 0, 0), np.float32),
                      np.zeros((L, H, 0, d), np.float32), np.zeros((L, H, 0, d), np.float32), n_cov=0)
    orc.apply(src, empty, 0, orc.rope_inv_freq(d, 10000.0), dst=dst)
    for l in range(L):
        for h in range(H):
            for t in range(T):
                assert np.array_equal(dst.k[l, pt_dst[t // page], h, t % page], code[l, h, t])
                assert np.array_equal(dst.v[l, pt_dst[t // page], h, t % page], code[l, h, t] ^ 0x4000)
    mapped = set(int(p) for p in pt_dst)
    for p in range(P):
        if p not in mapped:
            assert np.all(dst.k[:, p] == 0xBEEF) and np.all(dst.v[:, p] == 0xBEEF)
    # rows of the last, partial page beyond T are not written either
    tail = T % page
    assert np.all(dst.k[:, pt_dst[-1], :, tail:] == 0xBEEF)
