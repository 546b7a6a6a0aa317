"""Pins for the oracle's bf16 codec and RoPE re-alignment.

Nothing here re-types the oracle's own formula: the codec is checked against
torch's bfloat16 conversion and hand-worked roundings; the rotation against
the textbook 2x2 rotation, group properties and norm preservation.
"""
import math

import numpy as np
import torch

from oracle import kvc_oracle as orc


def test_bf16_widen_matches_torch():
    bits = np.arange(0, 65536, dtype=np.uint16)
    ours = orc.bf16_to_f64(bits)
    ref = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    finite = np.isfinite(ref)
    assert np.array_equal(ours[finite], ref[finite])
    assert np.array_equal(np.isnan(ours), np.isnan(ref))


def test_bf16_round_matches_torch_on_float32_inputs():
    rng = np.random.default_rng(0)
    x32 = np.concatenate([
        rng.standard_normal(200000).astype(np.float32),
        (rng.standard_normal(50000) * 1e-38).astype(np.float32),      # subnormal bf16 range
        (rng.standard_normal(50000) * 1e30).astype(np.float32),
        np.array([0.0, -0.0, 1.0, -1.0, 3.3895314e38, -3.3895314e38, 3.4e38, np.inf, -np.inf], np.float32),
    ])
    ours = orc.f64_to_bf16_bits(x32.astype(np.float64))
    ref = torch.from_numpy(x32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, ref)


def test_bf16_round_hand_cases():
    # spacing of bf16 in [1, 2) is 2^-7
    assert orc.round_to_bf16(1.0 + 2.0 ** -8) == 1.0                    # tie -> even (1.0)
    assert orc.round_to_bf16(1.0 + 2.0 ** -7 + 2.0 ** -8) == 1.0 + 2.0 ** -6  # tie -> even (up)
    # one rounding straight from float64: a hair above the tie must go up, although
    # rounding through float32 first would land on the tie and go down
    assert orc.round_to_bf16(1.0 + 2.0 ** -8 + 2.0 ** -40) == 1.0 + 2.0 ** -7
    assert orc.round_to_bf16(1.0 + 2.0 ** -8 - 2.0 ** -40) == 1.0
    # sign of zero survives
    assert math.copysign(1.0, float(orc.round_to_bf16(-0.0))) == -1.0
    assert orc.f64_to_bf16_bits(np.array([-0.0]))[0] == 0x8000
    # round trip of every finite pattern
    bits = np.arange(0, 65536, dtype=np.uint16)
    vals = orc.bf16_to_f64(bits)
    ok = np.isfinite(vals)
    assert np.array_equal(orc.f64_to_bf16_bits(vals[ok]), bits[ok])


def test_inv_freq_endpoints():
    f = orc.rope_inv_freq(128, 500000.0)
    assert f.shape == (64,)
    assert f[0] == 1.0
    # f_k is geometric with ratio theta^(-2/d); the last one is theta^(-(d-2)/d)
    assert np.allclose(f[1:] / f[:-1], 500000.0 ** (-2.0 / 128), rtol=1e-13)
    assert math.isclose(f[-1], 500000.0 ** (-126.0 / 128), rel_tol=1e-13)


def test_rope_d2_is_textbook_rotation():
    # d = 2: one pair, f_0 = 1, so Rot_s is the plane rotation by s radians
    x = np.array([[0.3, -1.7]])
    for s in (1, -3, 17):
        y = orc.rope_shift(x, s, orc.rope_inv_freq(2, 12345.0))
        R = np.array([[math.cos(s), -math.sin(s)], [math.sin(s), math.cos(s)]])
        assert np.allclose(y[0], R @ x[0], atol=1e-15)
    # quarter turn with an explicit frequency table: (1, 0) -> (0, 1)
    y = orc.rope_shift(np.array([[1.0, 0.0]]), 1, np.array([math.pi / 2]))
    assert np.allclose(y, [[0.0, 1.0]], atol=1e-15)


def test_rope_pairing_layouts():
    # one active pair at index k: half layout touches (k, k+d/2), interleaved (2k, 2k+1)
    d, k = 8, 2
    f = np.zeros(d // 2)
    f[k] = math.pi / 2
    x = np.arange(1.0, d + 1.0)[None, :]
    yh = orc.rope_shift(x, 1, f, orc.ROPE_HALF)[0]
    exp = x[0].copy()
    exp[k], exp[k + d // 2] = -x[0, k + d // 2], x[0, k]
    assert np.allclose(yh, exp, atol=1e-14)
    yi = orc.rope_shift(x, 1, f, orc.ROPE_INTERLEAVED)[0]
    exp = x[0].copy()
    exp[2 * k], exp[2 * k + 1] = -x[0, 2 * k + 1], x[0, 2 * k]
    assert np.allclose(yi, exp, atol=1e-14)


def test_rope_group_properties():
    rng = np.random.default_rng(1)
    d = 64
    f = orc.rope_inv_freq(d, 10000.0)
    x = rng.standard_normal((37, d))
    # shift 0 is the identity: the very same object, no arithmetic
    assert orc.rope_shift(x, 0, f) is x
    for a, b in ((16, 480), (-7, 7), (300, -512)):
        ab = orc.rope_shift(orc.rope_shift(x, a, f), b, f)
        assert np.allclose(ab, orc.rope_shift(x, a + b, f) if a + b else x, atol=1e-12)
    # inverse
    assert np.allclose(orc.rope_shift(orc.rope_shift(x, 123, f), -123, f), x, atol=1e-12)
    # each pair keeps its norm; the whole row too
    y = orc.rope_shift(x, 77, f)
    assert np.allclose(x[:, :32] ** 2 + x[:, 32:] ** 2, y[:, :32] ** 2 + y[:, 32:] ** 2, rtol=1e-12)
    # and the rotation really moves things (guards against a no-op implementation)
    assert np.max(np.abs(y - x)) > 0.5


def test_rope_preserves_dot_products_at_equal_shift():
    # attention scores between a query and a key moved by the same shift do not change
    rng = np.random.default_rng(2)
    d = 128
    f = orc.rope_inv_freq(d, 500000.0)
    q, k = rng.standard_normal((5, d)), rng.standard_normal((5, d))
    s = 211
    assert np.allclose(np.sum(orc.rope_shift(q, s, f) * orc.rope_shift(k, s, f), -1), np.sum(q * k, -1), atol=1e-11)


def test_per_token_shifts_equal_constant_shifts_segment_by_segment():
    """Multi-segment contexts (Eq. 1): rotating with a per-token shift vector is rotating every segment
    by its own constant shift; the segmented apply is the plain apply segment by segment; and the two
    coordinate conventions differ exactly by the rotation of the correction."""
    rng = np.random.default_rng(31)
    T, d, r = 37, 16, 3
    f = orc.rope_inv_freq(d, 10000.0)
    t_begin, shift = [0, 9, 20], [5, 0, -13]
    s_tok = orc.segment_shifts(T, t_begin, shift)
    assert s_tok.tolist() == [5] * 9 + [0] * 11 + [-13] * 17
    x = rng.standard_normal((T, d))
    for pairing in (orc.ROPE_HALF, orc.ROPE_INTERLEAVED):
        y = orc.rope_shift_tokens(x, s_tok, f, pairing)
        for j, t0 in enumerate(t_begin):
            t1 = t_begin[j + 1] if j + 1 < len(t_begin) else T
            assert np.array_equal(y[t0:t1], np.asarray(orc.rope_shift(x[t0:t1], shift[j], f, pairing)))
        # a scalar re-derivation of one element: pair (k, k + d/2) or (2k, 2k+1) turned by s f_k
        t, k = 30, 2
        i, j2 = (k, k + d // 2) if pairing == orc.ROPE_HALF else (2 * k, 2 * k + 1)
        ang = -13 * f[k]
        assert math.isclose(y[t, i], x[t, i] * math.cos(ang) - x[t, j2] * math.sin(ang), rel_tol=1e-12, abs_tol=1e-15)
        assert math.isclose(y[t, j2], x[t, i] * math.sin(ang) + x[t, j2] * math.cos(ang), rel_tol=1e-12, abs_tol=1e-15)
    # apply: segment by segment with the plain apply_slab (TARGET coordinates)
    bits = orc.f64_to_bf16_bits(x)
    c, B = rng.standard_normal((T, r)), rng.standard_normal((r, d))
    n_cov = 29
    ref, out = orc.apply_slab_tokens(bits, c, B, s_tok, f, n_cov, True)
    for j, t0 in enumerate(t_begin):
        t1 = t_begin[j + 1] if j + 1 < len(t_begin) else T
        n_seg = max(0, min(n_cov, t1) - t0)
        ref_j, out_j = orc.apply_slab(bits[t0:t1], c[t0:t1], B, shift[j], f, n_seg, True)
        assert np.array_equal(ref[t0:t1], ref_j) and np.array_equal(out[t0:t1], out_j)
    # values ignore the shifts; uncovered unshifted key rows keep their bits
    ref_v, out_v = orc.apply_slab_tokens(bits, c, B, s_tok, f, n_cov, False)
    ref_v0, out_v0 = orc.apply_slab(bits, c, B, 0, f, n_cov, False)
    assert np.array_equal(ref_v, ref_v0) and np.array_equal(out_v, out_v0)
    # SOURCE coordinates: the correction is rotated with the token; equal to TARGET with the rotated correction
    ref_s, _ = orc.apply_slab_tokens(bits, c, B, s_tok, f, T, True, coords=orc.COORDS_SOURCE)
    rotated_corr = orc.rope_shift_tokens(c @ B, s_tok, f)
    assert np.allclose(ref_s, orc.rope_shift_tokens(orc.bf16_to_f64(bits), s_tok, f) + rotated_corr, atol=1e-12)
    # with one shift for all tokens this is the re-aligned basis of App. A.2
    one = orc.segment_shifts(T, [0], [7])
    ref_1, _ = orc.apply_slab_tokens(bits, c, B, one, f, T, True, coords=orc.COORDS_SOURCE)
    ref_2, _ = orc.apply_slab(bits, c, orc.realign_basis(B, 7, f), 7, f, T, True)
    assert np.allclose(ref_1, ref_2, atol=1e-12)
    # deviations: SOURCE is TARGET carried back by the inverse rotation; fitting either reproduces the target
    tgt_bits = orc.f64_to_bf16_bits(rng.standard_normal((T, d)))
    d_t = orc.deviation_tokens(bits, tgt_bits, s_tok, f, True)
    d_s = orc.deviation_tokens(bits, tgt_bits, s_tok, f, True, coords=orc.COORDS_SOURCE)
    assert np.allclose(orc.rope_shift_tokens(d_s, s_tok, f), d_t, atol=1e-12)
    assert np.allclose(orc.rope_shift_tokens(orc.bf16_to_f64(bits) + d_s, s_tok, f), orc.bf16_to_f64(tgt_bits), atol=1e-12)
