"""Pins for the oracle's number formats and the group quantizer.

Every check compares the oracle with something that is not the oracle: values the
paper prints, independent library conversions (ml_dtypes / torch float8), exact
rational brute force, or invariants the format forces.
"""
import os
from fractions import Fraction

import ml_dtypes
import numpy as np
import pytest
import torch

import oracle
from paper_2411_09909_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_example.txt")
E2M1_SET = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]


def _golden():
    out = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        name, *vals = line.split()
        out[name] = [float(v) for v in vals]
    return out


def _fakequant(x64, gs):
    code4, scales = oracle.quantize_f64(x64, gs)
    return oracle.dequantize(oracle.pack_codes(code4), scales, gs)


# ------------------------------------------------------------ paper example --

@pytest.mark.parametrize("as_bf16", [False, True])
def test_worked_example_value_sets(as_bf16):
    """Appendix B.3: the three printed unique() sets, for fp32 and for bf16-cast input."""
    x = torch.linspace(-4.9, 31, 1024, dtype=torch.float32)
    if as_bf16:
        x = x.to(torch.bfloat16).float()
    x = x.double().numpy()[None, :]
    gold = _golden()
    assert sorted(set(_fakequant(x, 1024).ravel())) == gold["amxfp4_fp8"]
    assert sorted(set(oracle.fakequant_pot_floor(x, 1024, asym=False).ravel())) == gold["mxfp4_pot"]
    assert sorted(set(oracle.fakequant_pot_floor(x, 1024, asym=True).ravel())) == gold["amxfp4_pot"]


def test_worked_example_scales_and_extremes():
    """Appendix B.3 prose: 31 -> 30 under the FP8 scale (24 under PoT); scales 5.0 and 0.875."""
    x = torch.linspace(-4.9, 31, 1024).double().numpy()[None, :]
    code4, scales = oracle.quantize_f64(x, 1024)
    assert oracle.e5m2_value(scales[0, 0, 0]) == 5.0      # 31/6 = 5.1667 -> 1.25 * 2^2
    assert oracle.e5m2_value(scales[0, 0, 1]) == 0.875    # 4.9/6 = 0.8167 -> 1.75 * 2^-1
    deq = oracle.dequantize(oracle.pack_codes(code4), scales, 1024)
    assert deq[0, -1] == 30.0 and deq[0, 0] == -5.25
    assert oracle.fakequant_pot_floor(x, 1024, asym=False)[0, -1] == 24.0


# ------------------------------------------------------------------- E2M1 ----

def test_e2m1_decode_matches_ml_dtypes():
    """All 16 codes against an independent FP4 E2M1 implementation (sign in bit 3)."""
    lib_vals = np.arange(16, dtype=np.uint8).view(ml_dtypes.float4_e2m1fn).astype(np.float64)
    for c in range(16):
        assert oracle.e2m1_value(c) == lib_vals[c]
    # Eq. 1 element term: (-1)^s * 2^(E - 1) * (1 + M/2) for E > 0, M/2 for E = 0
    for c in range(16):
        s, E, M = c >> 3, (c >> 1) & 3, c & 1
        v = (2.0 ** (E - 1)) * (1 + M / 2) if E else M / 2
        assert oracle.e2m1_value(c) == (-v if s else v)


def test_e2m1_encode_matches_ml_dtypes_and_bruteforce():
    rng = np.random.default_rng(1)
    r = np.concatenate([rng.uniform(0, 8, 4000), np.arange(0, 32) / 4.0, [6.0, 6.5, 100.0, 1e30]])
    lib_codes = np.minimum(r, 6.0).astype(np.float32).astype(ml_dtypes.float4_e2m1fn).view(np.uint8)
    for ri, lc in zip(r, lib_codes):
        got = oracle.e2m1_encode(ri)
        assert got == int(lc), (ri, got, lc)
        # exact nearest search, ties to the even code
        d = [abs(Fraction(ri) - Fraction(m)) for m in E2M1_SET]
        best = min(d)
        cands = [k for k in range(8) if d[k] == best]
        want = cands[0] if len(cands) == 1 else [k for k in cands if k % 2 == 0][0]
        assert got == want


def test_e2m1_ties_go_to_even_code():
    for tie, want in [(0.25, 0.0), (0.75, 1.0), (1.25, 1.0), (1.75, 2.0), (2.5, 2.0), (3.5, 4.0), (5.0, 4.0)]:
        assert E2M1_SET[oracle.e2m1_encode(tie)] == want


# ------------------------------------------------------------------- E5M2 ----

def test_e5m2_decode_matches_torch_and_ml_dtypes():
    codes = np.arange(0, 0x7C, dtype=np.uint8)            # all finite non-negative codes
    tv = torch.from_numpy(codes.copy()).view(torch.float8_e5m2).double().numpy()
    mv = codes.view(ml_dtypes.float8_e5m2).astype(np.float64)
    for c in codes:
        assert oracle.e5m2_value(int(c)) == tv[c] == mv[c]
    assert oracle.e5m2_value(0x7B) == 57344.0
    assert oracle.e5m2_value(0x01) == 2.0 ** -16


def test_e5m2_encode_all_bf16_maxima_over_six():
    """scale = nearest E5M2 of max/6 for EVERY positive finite bf16 max, against exact
    rational nearest-value search over the 124 finite codes (ties -> even code, saturating)."""
    vals = [Fraction(oracle.e5m2_value(c)) for c in range(0x7C)]
    bits = np.arange(1, 0x7F80, dtype=np.uint16)
    maxima = inputs.bf16_bits_to_f32(bits).astype(np.float64)
    import bisect
    for mx in maxima[:: 7].tolist() + maxima[-40:].tolist() + [6.75, 27.0, 13.5, 6.0 * 2.0 ** -17]:
        q = Fraction(mx) / 6
        i = bisect.bisect_left(vals, q)
        if i == 0:
            want = 0
        elif i >= len(vals):
            want = 0x7B
        else:
            lo, hi = vals[i - 1], vals[i]
            if q - lo < hi - q:
                want = i - 1
            elif q - lo > hi - q:
                want = i
            else:
                want = i if i % 2 == 0 else i - 1
        assert oracle.e5m2_encode(mx / 6.0) == want, (mx, want)


def test_e5m2_encode_matches_library_in_range():
    rng = np.random.default_rng(2)
    q = np.exp2(rng.uniform(-19, 15.7, 20000)).astype(np.float32)
    tq = torch.from_numpy(q).to(torch.float8_e5m2).view(torch.uint8).numpy()
    mq = q.astype(ml_dtypes.float8_e5m2).view(np.uint8)
    for qi, a, b in zip(q.tolist(), tq.tolist(), mq.tolist()):
        got = oracle.e5m2_encode(qi)
        assert got == a == b, (qi, got, a, b)
    assert oracle.e5m2_encode(1e9) == 0x7B                 # saturates, never Inf
    assert oracle.e5m2_encode(0.0) == 0
    assert oracle.e5m2_encode(2.0 ** -18) == 0             # below half the smallest subnormal
    assert oracle.e5m2_encode(2.0 ** -17) == 0             # tie between 0 and 2^-16 -> even (0)
    assert oracle.e5m2_encode(3 * 2.0 ** -17) == 2         # tie between codes 1 and 2 -> even


# ---------------------------------------------------------- group quantizer --

def _decode(code4, scales, gs):
    return oracle.dequantize(oracle.pack_codes(code4), scales, gs)


def test_bruteforce_nearest_on_tiny_groups():
    """For the oracle's own scales each code must be the exact nearest of the 8 magnitudes of its
    side (ties -> even code), and each scale the exact nearest E5M2 of max_side/6."""
    rng = np.random.default_rng(3)
    e5 = [Fraction(oracle.e5m2_value(c)) for c in range(0x7C)]
    for gs in range(2, 9):
        x = rng.integers(-96, 97, size=(200, gs)).astype(np.float64) / 16.0
        x[rng.random(x.shape) < 0.1] = 0.0
        code4, scales = oracle.quantize_f64(x, gs)
        for r in range(x.shape[0]):
            row = [Fraction(v) for v in x[r]]
            neg = [np.signbit(v) for v in x[r]]
            for side in (0, 1):
                members = [abs(v) for v, n in zip(row, neg) if n == bool(side)]
                q = max(members, default=Fraction(0)) / 6
                d = [abs(q - v) for v in e5]
                best = min(d)
                cands = [c for c in range(0x7C) if d[c] == best]
                want = cands[0] if len(cands) == 1 else [c for c in cands if c % 2 == 0][0]
                assert scales[r, 0, side] == want
            for i in range(gs):
                s = e5[scales[r, 0, int(neg[i])]]
                c = int(code4[r, i])
                assert (c >> 3) == int(neg[i])
                if s == 0:
                    assert c & 7 == 0
                    continue
                d = [abs(abs(row[i]) - Fraction(m) * s) for m in E2M1_SET]
                best = min(d)
                cands = [k for k in range(8) if d[k] == best]
                want = cands[0] if len(cands) == 1 else [k for k in cands if k % 2 == 0][0]
                assert (c & 7) == want, (gs, r, i, x[r], c)


def test_side_extreme_maps_to_largest_code():
    """With a normal, unsaturated scale the largest element of each side encodes to +-6."""
    x = inputs.bf16_bits_to_f32(inputs.random_groups(11, 64, 256, "wide")).astype(np.float64)
    code4, scales = oracle.quantize_f64(x, 32)
    g = x.reshape(64, 8, 32)
    c = code4.reshape(64, 8, 32)
    for r in range(64):
        for j in range(8):
            for side, sel in ((0, ~np.signbit(g[r, j])), (1, np.signbit(g[r, j]))):
                sc = scales[r, j, side]
                if not sel.any():
                    assert sc == 0
                    continue
                if 4 <= sc < 0x7B:                           # normal and not saturated
                    k = np.argmax(np.where(sel, np.abs(g[r, j]), -1.0))
                    assert c[r, j, k] == (side << 3) | 7


def test_negation_swaps_scales_and_flips_signs():
    bits = inputs.random_groups(12, 32, 128, "mixed")
    c1, s1 = oracle.quantize(bits, 32)
    c2, s2 = oracle.quantize(bits ^ np.uint16(0x8000), 32)
    assert np.array_equal(c2, c1 ^ np.uint8(0x88))
    assert np.array_equal(s2, s1[:, :, ::-1])


def test_symmetric_group_reduces_to_single_scale_format():
    """pmax == nmax: both scales coincide and magnitudes equal those of quantizing |x| (the
    symmetric E2M1 + FP8-scale format the paper calls MXFP4 in its experiments, Section 5)."""
    rng = np.random.default_rng(4)
    x = rng.standard_normal((50, 32))
    x[:, 0] = np.abs(x).max(axis=1) * 1.5
    x[:, 1] = -x[:, 0]
    c, s = oracle.quantize_f64(x, 32)
    ca, sa = oracle.quantize_f64(np.abs(x), 32)
    assert np.array_equal(s[:, :, 0], s[:, :, 1])
    assert np.array_equal(s[:, :, 0], sa[:, :, 0])
    assert np.array_equal(c & 7, ca & 7)
    assert np.array_equal(c >> 3, np.signbit(x).astype(np.uint8))


def test_power_of_two_rescaling_shifts_scale_exponent_only():
    bits = inputs.random_groups(13, 16, 128, "normal")
    x = inputs.bf16_bits_to_f32(bits).astype(np.float64)
    c0, s0 = oracle.quantize_f64(x, 32)
    for k in (-9, 5):
        c1, s1 = oracle.quantize_f64(x * 2.0 ** k, 32)
        assert np.array_equal(c1, c0)
        assert np.array_equal(s1.astype(int), s0.astype(int) + 4 * k)


def test_roundtrip_of_all_codes_under_both_scales():
    """Decode every code under every pair of scales, re-encode: same codes, same scales, as long
    as each side holds a +-6 (so that the side maximum reproduces its scale)."""
    codes_all = np.arange(16, dtype=np.uint8)
    for sp in range(1, 0x7C, 5):
        for sn in range(2, 0x7C, 7):
            scales = np.array([[[sp, sn]]], np.uint8)
            code4 = np.concatenate([codes_all, [7, 15], np.zeros(14, np.uint8)])[None, :].astype(np.uint8)
            x = _decode(code4, scales, 32)
            c2, s2 = oracle.quantize_f64(x, 32)
            # decode drops the sign of zero magnitudes only when the value is +0; compare values
            assert np.array_equal(s2, scales)
            assert np.array_equal(_decode(c2, s2, 32), x)
            assert np.array_equal(c2 & 7, code4 & 7)


def test_quantization_error_bound():
    """|x - xhat| <= scale inside the grid (largest half-gap of E2M1 is 1) and <= 0.75*scale at the
    clamp (max/scale <= 6.75 after rounding the scale to 2 mantissa bits)."""
    bits = inputs.random_groups(14, 64, 256, "wide")
    x = inputs.bf16_bits_to_f32(bits).astype(np.float64)
    codes, scales = oracle.quantize(bits, 32)
    xh = oracle.dequantize(codes, scales, 32)
    sv = np.vectorize(oracle.e5m2_value)(scales).astype(np.float64)
    s_el = np.where(np.signbit(x).reshape(64, 8, 32), sv[:, :, 1:2], sv[:, :, 0:1]).reshape(64, 256)
    ok = np.repeat((scales >= 4) & (scales < 0x7B), 1, axis=2)
    ok_el = np.where(np.signbit(x).reshape(64, 8, 32), ok[:, :, 1:2], ok[:, :, 0:1]).reshape(64, 256)
    err = np.abs(x - xh)
    assert np.all(err[ok_el] <= s_el[ok_el] * (1 + 1e-12))
    assert np.all(np.sign(xh[xh != 0]) == np.sign(x[xh != 0]))


def test_empty_side_zero_group_and_negative_zero():
    x = np.zeros((1, 64))
    x[0, :32] = np.linspace(0.1, 3.0, 32)        # no negative members
    x[0, 40] = -0.0                              # second group: all zero, one negative zero
    c, s = oracle.quantize_f64(x, 32)
    assert s[0, 0, 1] == 0 and s[0, 1, 0] == 0 and s[0, 1, 1] == 0
    assert np.all(c[0, 32:] & 7 == 0)
    assert c[0, 40] == 8                         # sign bit kept on a zero magnitude
    assert np.all(oracle.dequantize(oracle.pack_codes(c), s, 32)[0, 32:] == 0.0)


def test_packing_layout_low_nibble_is_even_element():
    bits = inputs.random_groups(15, 4, 64, "normal")
    codes, scales = oracle.quantize(bits, 32)
    code4, scales2 = oracle.quantize_f64(inputs.bf16_bits_to_f32(bits).astype(np.float64), 32)
    assert np.array_equal(scales, scales2)
    assert np.array_equal(codes & 15, code4[:, 0::2])
    assert np.array_equal(codes >> 4, code4[:, 1::2])


def test_asymmetric_beats_symmetric_on_skewed_groups():
    """Direction of the paper's MSE comparison (Table of cluster-wise MSE: AsymFP4 < FP4)."""
    x = inputs.bf16_bits_to_f32(inputs.activation(3, 0, M=64)).astype(np.float64)   # SiLU-skewed
    xa = _fakequant(x, 32)
    # symmetric single-scale variant built from the same oracle: mirror each group so that both
    # sides share the group's absolute maximum
    g = x.reshape(-1, 32)
    amax = np.abs(g).max(axis=1, keepdims=True)
    gm = np.concatenate([g, amax, -amax], axis=1)
    c, s = oracle.quantize_f64(np.pad(gm, ((0, 0), (0, 30))), 64)
    xs = oracle.dequantize(oracle.pack_codes(c), s, 64)[:, :32].reshape(x.shape)
    assert np.mean((x - xa) ** 2) < np.mean((x - xs) ** 2)
