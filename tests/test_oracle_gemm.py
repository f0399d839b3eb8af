"""Pins for the oracle's dequantize, matrix product and softmax step."""
from fractions import Fraction

import ml_dtypes
import numpy as np
import scipy.special
import torch

import oracle
from paper_2411_09909_b200 import inputs


def _operands(seed, M, N, K, kind="mixed"):
    a = inputs.random_groups(seed, M, K, kind)
    w = inputs.random_groups(seed + 1, N, K, "normal")
    return oracle.quantize(a, 32), oracle.quantize(w, 32)


def _library_decode(codes, scales, gs=32):
    """Eq. 1 evaluated with independent library decoders (ml_dtypes FP4 / FP8)."""
    c4 = oracle.unpack_codes(codes)
    elem = c4.view(ml_dtypes.float4_e2m1fn).astype(np.float64)
    sv = scales.view(ml_dtypes.float8_e5m2).astype(np.float64)      # [rows, G, 2]
    side = (c4 >> 3).reshape(c4.shape[0], -1, gs)
    s_el = np.where(side == 1, sv[:, :, 1:2], sv[:, :, 0:1]).reshape(c4.shape)
    return elem * s_el


def test_dequantize_is_eq1_with_library_decoders():
    (ca, sa), _ = _operands(21, 24, 8, 256)
    assert np.array_equal(oracle.dequantize(ca, sa, 32), _library_decode(ca, sa))


def test_dequantized_values_fit_bf16_exactly():
    """E2M1 (2 significant bits) x E5M2 (3 significant bits) <= 5 significant bits."""
    (ca, sa), _ = _operands(22, 16, 8, 128, "wide")
    d = oracle.dequantize(ca, sa, 32)
    assert np.array_equal(d.astype(np.float32).astype(ml_dtypes.bfloat16).astype(np.float64), d)


def test_gemm_equals_fp64_matmul_of_decoded_operands():
    (ca, sa), (cw, sw) = _operands(23, 40, 72, 320)       # M != N != K catches a transposed operand
    ref = (_library_decode(ca, sa) @ _library_decode(cw, sw).T)
    got = oracle.gemm(ca, sa, cw, sw, 32)
    assert got.shape == (40, 72) and got.dtype == np.float32
    assert np.allclose(got, ref, rtol=1e-6, atol=0)
    # same sums in another order differ by fp64 rounding only
    assert np.max(np.abs(got - ref.astype(np.float32))) <= 4 * np.finfo(np.float32).eps * np.max(np.abs(ref))


def test_gemm_is_the_sign_selected_group_mac():
    """Section 4.3 / Fig. 5(b): per group the E2M1 products are summed per sign combination and
    each partial sum is multiplied by the product of the two shared scales those signs select.
    Evaluated in exact rational arithmetic from codes and scale bytes only."""
    (ca, sa), (cw, sw) = _operands(24, 6, 5, 96)
    a4, w4 = oracle.unpack_codes(ca), oracle.unpack_codes(cw)
    mag = [Fraction(0), Fraction(1, 2), Fraction(1), Fraction(3, 2), Fraction(2), Fraction(3), Fraction(4), Fraction(6)]
    e5 = [Fraction(float(np.uint8(c).view(ml_dtypes.float8_e5m2))) for c in range(0x7C)]
    got = oracle.gemm(ca, sa, cw, sw, 32)
    for m in range(6):
        for n in range(5):
            total = Fraction(0)
            for g in range(3):
                part = {(0, 0): Fraction(0), (0, 1): Fraction(0), (1, 0): Fraction(0), (1, 1): Fraction(0)}
                for k in range(32 * g, 32 * g + 32):
                    a, w = int(a4[m, k]), int(w4[n, k])
                    sign = -1 if ((a >> 3) ^ (w >> 3)) else 1
                    part[(a >> 3, w >> 3)] += sign * mag[a & 7] * mag[w & 7]
                for (sa_side, sw_side), p in part.items():
                    total += p * e5[sa[m, g, sa_side]] * e5[sw[n, g, sw_side]]
            assert got[m, n] == np.float32(float(total)), (m, n)


def test_gemm_exact_on_dyadic_inputs_and_row_selection():
    rng = np.random.default_rng(5)
    a = rng.integers(-6, 7, size=(64, 128)).astype(np.float32)
    w = rng.integers(-6, 7, size=(48, 128)).astype(np.float32)
    a[:, ::32] = 6.0; a[:, 1::32] = -6.0                   # scales exactly 1: codes hold the integers
    w[:, ::32] = 6.0; w[:, 1::32] = -6.0
    grid = np.array([0, 1, 2, 3, 4, 6], np.float32)
    snap = lambda t: np.sign(t) * grid[np.abs(np.abs(t)[..., None] - grid).argmin(-1)]
    a, w = snap(a), snap(w)
    qa = oracle.quantize(inputs.f32_to_bf16_bits(a), 32)
    qw = oracle.quantize(inputs.f32_to_bf16_bits(w), 32)
    assert np.array_equal(oracle.dequantize(*qa, 32), a.astype(np.float64))
    ref = a.astype(np.int64) @ w.astype(np.int64).T
    assert np.array_equal(oracle.gemm(*qa, *qw, 32), ref.astype(np.float32))
    rows = np.array([63, 0, 17, 17], np.int64)
    assert np.array_equal(oracle.gemm(*qa, *qw, 32, rows=rows), ref[rows].astype(np.float32))


def test_softmax_bf16_against_scipy_and_torch_rounding():
    rng = np.random.default_rng(6)
    S = (rng.standard_normal((32, 300)) * 20).astype(np.float32)
    alpha = 128 ** -0.5
    ref = scipy.special.softmax(S.astype(np.float64) * alpha, axis=1)
    got = oracle.softmax_bf16(S, alpha)
    want = torch.from_numpy(ref).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    # identical except where the fp64 value sits within rounding error of a bf16 midpoint
    assert np.mean(got == want) > 0.999
    assert np.max(np.abs(got.astype(np.int32) - want.astype(np.int32))) <= 1
    p = inputs.bf16_bits_to_f32(got).astype(np.float64)
    assert np.allclose(p.sum(axis=1), 1.0, atol=2e-2)
    assert np.all(np.abs(p - ref) <= ref * 2.0 ** -8 + 1e-45)


def test_causal_softmax_is_the_masked_softmax():
    rng = np.random.default_rng(9)
    S = (rng.standard_normal((24, 40)) * 10).astype(np.float32)
    alpha = 0.25
    got = inputs.bf16_bits_to_f32(oracle.softmax_bf16(S, alpha, causal_row0=8)).astype(np.float64)
    masked = np.where(np.arange(40)[None, :] <= (np.arange(24)[:, None] + 8), S.astype(np.float64) * alpha, -np.inf)
    ref = scipy.special.softmax(masked, axis=1)
    assert np.all(got[np.isinf(masked)] == 0)
    assert np.all(np.abs(got - ref) <= ref * 2.0 ** -8 + 1e-45)
    # the first query (row0 = 0) sees one key only; rows that see every key equal the unmasked softmax
    first = oracle.softmax_bf16(S[:1], alpha, causal_row0=0)
    assert first[0, 0] == 0x3F80 and not first[0, 1:].any()
    assert np.array_equal(oracle.softmax_bf16(S, alpha, causal_row0=39), oracle.softmax_bf16(S, alpha))


def test_input_generators_are_seeded_and_shaped():
    a1, a2 = inputs.activation(2, 0, M=8), inputs.activation(2, 0, M=8)
    assert a1.dtype == np.uint16 and a1.shape == (8, 4096) and np.array_equal(a1, a2)
    assert inputs.weight(4, 2, N=4).shape == (4, 28672)
    q, k, v = inputs.attention_qkv(heads=2, seq=64)
    assert q.shape == k.shape == v.shape == (2, 64, 128) and not np.array_equal(q, k)
    a = inputs.bf16_bits_to_f32(inputs.activation(1, 0))
    assert (np.abs(a).max(axis=0) > 60).sum() == 10        # the ten outlier channels
    silu = inputs.bf16_bits_to_f32(inputs.activation(3, 0, M=16))
    assert silu.min() > -0.3                                # SiLU is bounded below at -0.2785
    x = np.array([1.00390625, 1.01171875, -3.0e38, 1e-40], np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(inputs.f32_to_bf16_bits(x), want)
