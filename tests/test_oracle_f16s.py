"""Pins of the oracle's FP4 quantizer with binary16 shared scales (the "FP16" row of the appendix's ablation of the
shared-scale encoding, symmetric and asymmetric) against things other than itself: numpy's binary16, exact rational
nearest-value search, the (separately pinned) FP8-scale quantizer where the two formats must agree, and invariants."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2411_09909_b200 import inputs

E2M1 = [Fraction(0), Fraction(1, 2), Fraction(1), Fraction(3, 2), Fraction(2), Fraction(3), Fraction(4), Fraction(6)]


def bits(x):
    return inputs.f32_to_bf16_bits(np.asarray(x, np.float32))


def values(b):
    return inputs.bf16_bits_to_f32(b).astype(np.float64)


def test_f16_value_and_encode_match_numpy():
    pat = np.arange(0x7C00, dtype=np.uint16)                       # every finite non-negative pattern
    lib_vals = pat.view(np.float16).astype(np.float64)
    assert all(oracle.f16_value(int(p)) == v for p, v in zip(pat[::7], lib_vals[::7]))
    assert oracle.f16_value(0x8001) == -2.0 ** -24 and oracle.f16_value(0x7BFF) == 65504.0
    rng = np.random.default_rng(11)
    q = np.concatenate([2.0 ** rng.uniform(-27, 16, 4000), rng.uniform(0, 2.0 ** -13, 2000),
                        (lib_vals[:-1] + lib_vals[1:])[::5] / 2,    # exact midpoints: ties to the even mantissa
                        lib_vals[::11], [2.0 ** -25, 2.0 ** -25 * 1.0000001, 65504.0, 65519.9]])
    got = np.array([oracle.f16_encode(v) for v in q], np.uint16)
    want = q.astype(np.float16).view(np.uint16)                    # numpy rounds float64 -> binary16 correctly
    assert np.array_equal(got, want)
    for big in (65520.0, 1e6, 1e30):                               # numpy gives inf there; the quantizer saturates
        assert oracle.f16_encode(big) == 0x7BFF
    assert oracle.f16_encode(0.0) == 0 and oracle.f16_encode(2.0 ** -26) == 0


def nearest_f16(q: Fraction) -> int:
    """binary16 pattern nearest to the rational q >= 0 by exact comparison with its neighbours (ties: even pattern)."""
    if q >= 65520:
        return 0x7BFF
    c = int(np.float16(float(q)).view(np.uint16))                  # a candidate; float(q) may be off by one ulp of fp64
    best = None
    for p in (c - 1, c, c + 1):
        if 0 <= p <= 0x7BFF:
            d = abs(Fraction(float(np.uint16(p).view(np.float16))) - q)
            if best is None or d < best[0] or (d == best[0] and p % 2 == 0):
                best = (d, p)
    return best[1]


def nearest_code(x: Fraction, s: Fraction) -> int:
    if s == 0:
        return 0
    r = min(abs(x) / s, Fraction(6))
    best = None
    for c, m in enumerate(E2M1):
        d = abs(r - m)
        if best is None or d < best[0] or (d == best[0] and c % 2 == 0):
            best = (d, c)
    return best[1]


@pytest.mark.parametrize("asym", [False, True])
@pytest.mark.parametrize("gs", [16, 32, 64, 128])
def test_exact_rational_search(gs, asym):
    """Scales and codes of small random tensors (wide range, one-sided and zero groups included) equal the nearest
    binary16 of max/6 and the nearest E2M1 of x/scale in exact rational arithmetic."""
    rng = np.random.default_rng(100 + gs + asym)
    rows, K = 5, 2 * gs
    x = rng.standard_normal((rows, K)) * 2.0 ** rng.integers(-20, 14, (rows, 1))
    x[0, :gs] = np.abs(x[0, :gs])                                   # one-sided
    x[1, gs:] = 0.0                                                 # all zero
    x[2, :gs] *= 2.0 ** -18                                         # binary16-subnormal scales
    x[3, 0] = 3.0e38                                                # scale saturates at 65504: everything clamps
    b = bits(x)
    v = values(b)
    codes, scales = oracle.quantize_f16s(b, gs, asym)
    c4 = oracle.unpack_codes(codes)
    for r in range(rows):
        for g in range(K // gs):
            seg, sb = v[r, g * gs:(g + 1) * gs], b[r, g * gs:(g + 1) * gs]
            neg = (sb >> 15).astype(bool)
            pmax = max([Fraction(float(a)) for a, n in zip(seg, neg) if not n], default=Fraction(0))
            nmax = max([Fraction(float(-a)) for a, n in zip(seg, neg) if n], default=Fraction(0))
            if not asym:
                pmax = nmax = max(pmax, nmax)
            want = (nearest_f16(pmax / 6), nearest_f16(nmax / 6))
            assert tuple(int(s) for s in scales[r, g]) == want
            sv = [Fraction(float(np.uint16(w).view(np.float16))) for w in want]
            for i in range(gs):
                s = sv[int(neg[i])]
                assert c4[r, g * gs + i] == (int(neg[i]) << 3 | nearest_code(Fraction(float(seg[i])), s))


def test_agrees_with_fp8_scale_quantizer_when_scales_are_representable():
    """Group maxima of the form 6 * (1, 1.25, 1.5 or 1.75) * 2^k have an E5M2 scale that is exact, hence the same
    scale in binary16: codes and decoded values of the two quantizers must then be identical."""
    rng = np.random.default_rng(12)
    rows, G, gs = 16, 4, 32
    x = rng.standard_normal((rows, G * gs)).astype(np.float32)
    for r in range(rows):
        for g in range(G):
            seg = x[r, g * gs:(g + 1) * gs]
            sp = (1 + rng.integers(0, 4) / 4) * 2.0 ** rng.integers(-10, 8)
            sn = (1 + rng.integers(0, 4) / 4) * 2.0 ** rng.integers(-10, 8)
            seg[:] = np.where(seg >= 0, seg / np.abs(seg).max() * 5.9 * sp, seg / np.abs(seg).max() * 5.9 * sn)
            seg[0], seg[1] = 6 * sp, -6 * sn
    b = bits(x)
    c8, s8 = oracle.quantize(b, gs)
    c16, s16 = oracle.quantize_f16s(b, gs, True)
    assert np.array_equal(c8, c16)
    v8 = np.vectorize(oracle.e5m2_value)(s8)
    v16 = s16.view(np.float16).astype(np.float64)
    assert np.array_equal(v8, v16)
    assert np.array_equal(oracle.dequantize(c8, s8, gs), oracle.dequantize_f16s(c16, s16, gs))


@pytest.mark.parametrize("asym", [False, True])
def test_invariants(asym):
    rng = np.random.default_rng(13 + asym)
    gs = 32
    x = (rng.standard_normal((12, 4 * gs)) * 2.0 ** rng.integers(-6, 6, (12, 1))).astype(np.float32)
    x[:, ::5] += 1.5                                                 # non-zero group means: the two sides differ
    b = bits(x)
    v = values(b)
    codes, scales = oracle.quantize_f16s(b, gs, asym)
    xhat = oracle.dequantize_f16s(codes, scales, gs)
    # negation swaps the two scales and flips every sign bit
    cn, sn = oracle.quantize_f16s(b ^ 0x8000, gs, asym)
    assert np.array_equal(sn, scales[:, :, ::-1])
    assert np.array_equal(oracle.unpack_codes(cn), oracle.unpack_codes(codes) ^ 8)
    # multiplying by a power of two (inside the binary16 range) multiplies scales and decoded values by it
    c2, s2 = oracle.quantize_f16s(bits(v * 8.0), gs, asym)
    assert np.array_equal(c2, codes)
    assert np.array_equal(oracle.dequantize_f16s(c2, s2, gs), xhat * 8.0)
    # a side's extreme decodes to +-6 * scale; nothing decodes beyond it; the symmetric format has one scale
    sv = scales.view(np.float16).astype(np.float64)
    if not asym:
        assert np.array_equal(scales[..., 0], scales[..., 1])
    g_of = np.arange(x.shape[1]) // gs
    side = (b >> 15).astype(int)
    s_el = sv[np.arange(12)[:, None], g_of[None, :], side]
    assert np.all(np.abs(xhat) <= 6.0 * s_el)
    # error bound: half the largest gap of the element grid (1 * scale), plus the clamp overshoot max - 6 * scale,
    # which the rounding of the scale bounds by 2^-11 relative
    assert np.all(np.abs(v - xhat) <= s_el * (1.0 + 6.0 * 2.0 ** -11) + 1e-300)
    # the finer scale cannot clamp by more than one binary16 rounding: |x| <= 6 * scale * (1 + 2^-11)
    assert np.all(np.abs(v) <= 6.0 * s_el * (1 + 2.0 ** -11))
    # each side's extreme element is reproduced to one binary16 rounding of its scale (the FP8 scale: 2^-3)
    for r in range(12):
        for g in range(x.shape[1] // gs):
            seg, hat = v[r, g * gs:(g + 1) * gs], xhat[r, g * gs:(g + 1) * gs]
            for ext in (seg.max(), seg.min()):
                if ext != 0 and (asym or abs(ext) == np.abs(seg).max()):
                    i = int(np.where(seg == ext)[0][0])
                    assert abs(hat[i] - ext) <= abs(ext) * 2.0 ** -11


def nearest_e4m3_as_f16(q: Fraction) -> int:
    """binary16 pattern of the FP8 E4M3 value nearest to q >= 0 (exact comparison over all 127 finite values; ties to
    the even E4M3 code; saturating at 448), with ml_dtypes as the table of E4M3 values."""
    import ml_dtypes
    vals = np.arange(0x7F, dtype=np.uint8).view(ml_dtypes.float8_e4m3fn).astype(np.float64)
    best = None
    for code, v in enumerate(vals):
        d = abs(Fraction(float(v)) - q)
        if best is None or d < best[0] or (d == best[0] and code % 2 == 0):
            best = (d, code)
    return int(np.float16(vals[best[1]]).view(np.uint16))


@pytest.mark.parametrize("asym", [False, True])
def test_e4m3_scale_option(asym):
    rng = np.random.default_rng(15 + asym)
    gs, rows, K = 32, 6, 128
    x = rng.standard_normal((rows, K)) * 2.0 ** rng.integers(-8, 9, (rows, 1))
    x[0, :gs] *= 2.0 ** -9                                           # E4M3-subnormal scales
    x[1, 0] = 1.0e5                                                  # saturates at 448: everything above 2688 clamps
    x[2, gs:2 * gs] = 0.0
    b = bits(x)
    v = values(b)
    codes, scales = oracle.quantize_f16s(b, gs, asym, e4m3=True)
    c4 = oracle.unpack_codes(codes)
    for r in range(rows):
        for g in range(K // gs):
            seg, sb = v[r, g * gs:(g + 1) * gs], b[r, g * gs:(g + 1) * gs]
            neg = (sb >> 15).astype(bool)
            pmax = max([Fraction(float(a)) for a, n in zip(seg, neg) if not n], default=Fraction(0))
            nmax = max([Fraction(float(-a)) for a, n in zip(seg, neg) if n], default=Fraction(0))
            if not asym:
                pmax = nmax = max(pmax, nmax)
            want = (nearest_e4m3_as_f16(pmax / 6), nearest_e4m3_as_f16(nmax / 6))
            assert tuple(int(s) for s in scales[r, g]) == want
            sv = [Fraction(float(np.uint16(w).view(np.float16))) for w in want]
            for i in range(gs):
                assert c4[r, g * gs + i] == (int(neg[i]) << 3 | nearest_code(Fraction(float(seg[i])), sv[int(neg[i])]))
    assert scales.view(np.float16).astype(np.float64).max() == 448.0
    # where the binary16 scale happens to be an E4M3 value the two options agree
    c16, s16 = oracle.quantize_f16s(b, gs, asym)
    same = (s16 == scales).all(axis=2)
    k = np.repeat(same, gs, axis=1)
    assert np.array_equal(oracle.unpack_codes(c16)[k], c4[k])


def test_gemm_and_error_sums():
    rng = np.random.default_rng(14)
    gs = 16
    # integer-valued operands whose group maxima are 6 (scale exactly 1): the product is an exact integer matrix
    A = rng.integers(-4, 5, (7, 64)).astype(np.float32)
    W = rng.integers(-4, 5, (9, 64)).astype(np.float32)
    A[A == 5] = 4; W[W == 5] = 4
    A[:, ::gs], A[:, 1::gs], W[:, ::gs], W[:, 1::gs] = 6, -6, 6, -6
    A[np.abs(A) == 0] = 0
    ca, sa = oracle.quantize_f16s(bits(A), gs, True)
    cw, sw = oracle.quantize_f16s(bits(W), gs, True)
    assert np.all(sa == 0x3C00) and np.all(sw == 0x3C00)            # binary16 1.0
    assert np.array_equal(oracle.dequantize_f16s(ca, sa, gs), A.astype(np.float64))
    assert np.array_equal(oracle.gemm_f16s(ca, sa, cw, sw, gs), (A.astype(np.int64) @ W.astype(np.int64).T).astype(np.float32))
    # general operands: the product of the dequantized matrices in numpy's fp64
    X = rng.standard_normal((6, 96)).astype(np.float32) * 3
    Y = rng.standard_normal((5, 96)).astype(np.float32) * 0.02
    cx, sx = oracle.quantize_f16s(bits(X), 32, False)
    cy, sy = oracle.quantize_f16s(bits(Y), 32, True)
    ref = oracle.dequantize_f16s(cx, sx, 32) @ oracle.dequantize_f16s(cy, sy, 32).T
    np.testing.assert_allclose(oracle.gemm_f16s(cx, sx, cy, sy, 32), ref, rtol=2e-7, atol=0)
    # error sums against numpy on the dequantized tensor; nothing clamps beyond one rounding of the scale
    bx = bits(X)
    out = oracle.quant_error_f16s(bx, cx, sx, 32)
    v, xh = values(bx), oracle.dequantize_f16s(cx, sx, 32)
    assert out[0] == pytest.approx((v * v).sum(), rel=1e-12) and out[1] == pytest.approx(((v - xh) ** 2).sum(), rel=1e-12)
    sv = sx.view(np.float16).astype(np.float64)
    s_el = sv[np.arange(6)[:, None], (np.arange(96) // 32)[None, :], (bx >> 15).astype(int)]
    clamped = np.abs(v) > 6 * s_el
    assert out[3] == clamped.sum() and out[2] == pytest.approx(((v - xh) ** 2)[clamped].sum(), rel=1e-12, abs=0)
