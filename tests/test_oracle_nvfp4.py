"""Pins of the oracle's NVFP4 / ANVFP4 quantizer (group 16, E4M3 group scales, one fp32 tensor scale: the format
the paper compares with in Section 5) against things other than itself: an independent E4M3 implementation,
exact rational arithmetic, closed forms and invariants of the format."""
from fractions import Fraction

import ml_dtypes
import numpy as np
import pytest

import oracle
from paper_2411_09909_b200 import inputs

E2M1 = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]


def bits(x):
    return inputs.f32_to_bf16_bits(np.asarray(x, np.float32))


def values(b):
    return inputs.bf16_bits_to_f32(b).astype(np.float64)


def test_e4m3_matches_ml_dtypes():
    lib_vals = np.arange(256, dtype=np.uint8).view(ml_dtypes.float8_e4m3fn).astype(np.float64)
    for c in range(256):
        v = oracle.e4m3_value(c)
        assert (np.isnan(v) and np.isnan(lib_vals[c])) or v == lib_vals[c]
    rng = np.random.default_rng(3)
    q = np.concatenate([rng.uniform(0, 500, 3000), rng.uniform(0, 0.05, 2000), 2.0 ** rng.uniform(-12, 9, 3000)])
    # every midpoint between neighbouring E4M3 values as well (ties go to the even mantissa)
    pos = np.sort(lib_vals[:0x7F])
    q = np.concatenate([q, (pos[:-1] + pos[1:]) / 2, pos, [448.0, 449.0, 464.0, 480.0, 1e6]])
    got = np.array([oracle.e4m3_encode(v) for v in q])
    want = np.minimum(q, 448.0).astype(np.float32).astype(ml_dtypes.float8_e4m3fn).view(np.uint8)
    assert np.array_equal(got, want)


def test_tensor_scale_and_top_of_range():
    """t = max|x| / 2688; the group holding the tensor's largest element gets the largest E4M3 scale (448) and that
    element the code 6; an all-zero tensor has t = 1 and zero codes and scales."""
    rng = np.random.default_rng(4)
    x = rng.standard_normal((8, 64)).astype(np.float32)
    x[3, 20] = -37.5
    b = bits(x)
    for asym in (False, True):
        codes, scales, t = oracle.quantize_nv(b, asym)
        assert t == np.float32(np.float32(37.5) / np.float32(2688.0))
        assert scales[3, 1, 1] == 0x7E                                   # group 1 of row 3, negative side: 448
        c = oracle.unpack_codes(codes)[3, 20]
        assert c == 0xF                                                   # -6
        assert oracle.dequantize_nv(codes, scales, t)[3, 20] == pytest.approx(-37.5, rel=2 ** -20)
    z = np.zeros((2, 32), np.uint16)
    codes, scales, t = oracle.quantize_nv(z, True)
    assert t == 1.0 and not codes.any() and not scales.any()


@pytest.mark.parametrize("asym", [False, True])
def test_exact_inputs_match_rational_nearest_search(asym):
    """Inputs for which every fp32 step of the reference is exact (tensor maximum 2688 * 2^k, so t is a power of
    two; group maxima 6 * an E4M3 value * t; elements on a grid of eighths of the scale): codes must be the nearest
    E2M1 value in exact rational arithmetic, ties to the even code."""
    rng = np.random.default_rng(5 + asym)
    rows, G = 6, 8
    t = 2.0 ** -3
    # normal E4M3 values with significand 1 or 1.5: a multiple of a quarter of such a scale, up to 24 quarters,
    # has at most 7 significant bits (exact in bf16), and the reciprocal multiply is exact at every tie
    e4 = [oracle.e4m3_value(c) for c in range(8, 0x7F) if (c & 7) in (0, 4)]
    x = np.zeros((rows, G * 16), np.float32)
    want_scale = np.zeros((rows, G, 2), np.uint8)
    for r in range(rows):
        for g in range(G):
            sp, sn = rng.choice(e4[:-1], 2)
            if not asym:
                sn = sp
            seg = x[r, g * 16:(g + 1) * 16]
            for i in range(16):
                neg = rng.random() < 0.5
                s = sn if neg else sp
                # multiples of s / 4 with a short significand: exact in bf16 when s has <= 4 significant bits
                m = int(rng.integers(0, 25))
                seg[i] = (-1 if neg else 1) * m * s * t / 4
            seg[0], seg[1] = 6 * sp * t, -6 * sn * t                      # the side maxima fix the scales
            want_scale[r, g] = [oracle.e4m3_encode(sp), oracle.e4m3_encode(sn)]
    x[0, 0] = 2688 * t                                                    # fixes the tensor scale (its group: scale 448)
    want_scale[0, 0, 0] = 0x7E
    if not asym:
        want_scale[0, 0, 1] = 0x7E
    b = bits(x)
    assert np.array_equal(values(b), x.astype(np.float64))               # the inputs are exact in bf16
    codes, scales, tt = oracle.quantize_nv(b, asym)
    assert tt == np.float32(t)
    assert np.array_equal(scales, want_scale)
    c4 = oracle.unpack_codes(codes)
    for r in range(rows):
        for k in range(G * 16):
            xv = Fraction(float(x[r, k]))
            neg = b[r, k] >> 15
            s = Fraction(oracle.e4m3_value(int(scales[r, k // 16, neg]))) * Fraction(t)
            q = abs(xv) / s
            best = min(range(8), key=lambda c: (abs(min(q, Fraction(6)) - Fraction(E2M1[c])), c & 1))
            assert c4[r, k] == (neg << 3 | best), (r, k)


@pytest.mark.parametrize("asym", [False, True])
def test_general_inputs_agree_with_exact_arithmetic_away_from_boundaries(asym):
    """Seeded general inputs: the fp32 decisions of the reference equal exact-rational decisions unless the exact
    quotient lies within 2^-20 (relative) of a rounding boundary."""
    b = inputs.random_groups(7, 12, 256, "normal")
    codes, scales, t = oracle.quantize_nv(b, asym)
    x = values(b)
    tq = Fraction(float(t))
    c4 = oracle.unpack_codes(codes)
    mids = [Fraction(v) for v in (0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0)]
    checked = 0
    for r in range(12):
        for g in range(16):
            seg = x[r, g * 16:(g + 1) * 16]
            neg = (b[r, g * 16:(g + 1) * 16] >> 15).astype(bool)
            pm = max([abs(v) for v, n in zip(seg, neg) if not n], default=0.0)
            nm = max([abs(v) for v, n in zip(seg, neg) if n], default=0.0)
            if not asym:
                pm = nm = max(pm, nm)
            for side, mx in ((0, pm), (1, nm)):
                exact = Fraction(mx) / 6 / tq
                want = oracle.e4m3_encode(float(exact))                  # fp64 is exact enough away from boundaries
                lo, hi = oracle.e4m3_value(max(want - 1, 0)), oracle.e4m3_value(min(want + 1, 0x7E))
                near = any(abs(float(exact) - (oracle.e4m3_value(want) + o) / 2) <= 2 ** -20 * float(exact) for o in (lo, hi))
                if not near:
                    assert scales[r, g, side] == want
            for i in range(16):
                s = Fraction(oracle.e4m3_value(int(scales[r, g, int(neg[i])]))) * tq
                if s == 0:
                    assert c4[r, g * 16 + i] & 7 == 0
                    continue
                q = min(abs(Fraction(float(seg[i]))) / s, Fraction(6))
                if any(abs(q - m) <= Fraction(1, 2 ** 20) * q for m in mids):
                    continue
                best = min(range(8), key=lambda c: (abs(q - Fraction(E2M1[c])), c & 1))
                assert c4[r, g * 16 + i] & 7 == best
                checked += 1
    assert checked > 2500


def test_format_invariants():
    b = inputs.random_groups(8, 20, 128, "normal")
    cA, sA, tA = oracle.quantize_nv(b, True)
    # negation swaps the two scales of every group and flips every sign bit
    cN, sN, tN = oracle.quantize_nv(b ^ 0x8000, True)
    assert tN == tA and np.array_equal(sN, sA[:, :, ::-1]) and np.array_equal(cN, cA ^ 0x88)
    # a power-of-two rescaling moves only the tensor scale
    scaled = bits(values(b) * 2.0 ** 5)
    cS, sS, tS = oracle.quantize_nv(scaled, True)
    assert tS == np.float32(tA * 32) and np.array_equal(cS, cA) and np.array_equal(sS, sA)
    # groups whose two sides have the same maximum: ANVFP4 = NVFP4 there
    sym = b.copy()
    sym[:, 0::16] = (sym[:, 0::16] & 0x807F) | 0x4100  # element 0 of each group: magnitude in [8, 16) ...
    sym[:, 1::16] = sym[:, 0::16] ^ 0x8000            # ... element 1 = minus element 0 ...
    big = (sym[:, 0::16] & 0x7FFF).astype(np.uint32)
    rest = (sym.reshape(20, 8, 16)[:, :, 2:] & 0x7FFF).max(axis=2)
    ok = big >= rest                                 # ... and it is the group's largest magnitude
    cY, sY, _ = oracle.quantize_nv(sym, True)
    cZ, sZ, _ = oracle.quantize_nv(sym, False)
    assert ok.sum() > 100
    assert np.array_equal(sY[ok], sZ[ok])
    assert np.array_equal(cY.reshape(20, 8, 8)[ok], cZ.reshape(20, 8, 8)[ok])
    # the side extreme maps to magnitude 6 whenever its scale is a normal, unsaturated E4M3 number
    c4 = oracle.unpack_codes(cA).reshape(20, 8, 16)
    x = values(b).reshape(20, 8, 16)
    for r in range(20):
        for g in range(8):
            for side in (0, 1):
                byte = sA[r, g, side]
                sel = (b.reshape(20, 8, 16)[r, g] >> 15) == side
                if 8 <= byte < 0x7E and sel.any():
                    i = np.argmax(np.where(sel, np.abs(x[r, g]), -1))
                    assert c4[r, g, i] & 7 == 7
    # error bound: inside the grid |x - xhat| <= scale (half the widest gap), beyond 6 the clamp loses <= 0.38 scale
    d = oracle.dequantize_nv(cA, sA, tA)
    side = (b >> 15).astype(int)
    s_el = np.vectorize(oracle.e4m3_value)(np.take_along_axis(np.repeat(sA, 16, axis=1), side[:, :, None], axis=2)[:, :, 0]) * float(tA)
    assert np.all(np.abs(values(b) - d) <= s_el * 1.0001)


def test_gemm_nv_is_the_decoded_product():
    a = inputs.random_groups(9, 10, 128, "normal")
    w = inputs.random_groups(10, 14, 128, "normal")
    qa, qw = oracle.quantize_nv(a, True), oracle.quantize_nv(w, False)
    ref = oracle.dequantize_nv(*qa) @ oracle.dequantize_nv(*qw).T
    got = oracle.gemm_nv(*qa, *qw)
    assert np.allclose(got, ref, rtol=1e-6, atol=0)
    rows = np.array([7, 2])
    assert np.array_equal(oracle.gemm_nv(*qa, *qw, rows=rows), got[rows])
