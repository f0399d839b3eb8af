"""Pins for the oracle's symmetric comparison formats (one shared scale per group)."""
import os

import ml_dtypes
import numpy as np

import oracle
from paper_2411_09909_b200 import inputs


def _bits(x):
    return inputs.f32_to_bf16_bits(np.asarray(x, np.float32))


def test_mxfp4_reproduces_the_printed_value_set():
    """Appendix B.3 prints the MXFP4 values of linspace(-4.9, 31, 1024) quantized as one group."""
    path = os.path.join(os.path.dirname(__file__), "golden", "worked_example.txt")
    printed = next(line.split()[1:] for line in open(path) if line.startswith("mxfp4_pot "))
    x = _bits(np.linspace(-4.9, 31, 1024, dtype=np.float32))[None, :]
    c, s = oracle.quantize_variant(x, 1024, oracle.MXFP4)
    got = np.unique(oracle.dequantize(c, s, 1024))
    assert got.tolist() == sorted(float(t) for t in printed)
    assert s[0, 0, 0] == s[0, 0, 1] and oracle.e5m2_value(int(s[0, 0, 0])) == 4.0     # 2^(floor(log2 31) - 2)


def test_mxfp4_equals_algorithm1_fake_quant():
    """Decoding the stored codes gives Algorithm 1's result (the fake-quant routine the printed sets pin)."""
    bits = inputs.random_groups(31, 64, 256, "normal")
    c, s = oracle.quantize_variant(bits, 32, oracle.MXFP4)
    x = inputs.bf16_bits_to_f32(bits).astype(np.float64)
    assert np.array_equal(oracle.dequantize(c, s, 32), oracle.fakequant_pot_floor(x, 32, asym=False))
    # the scale byte is a power of two read back by an independent decoder
    sv = s[..., 0].view(ml_dtypes.float8_e5m2).astype(np.float64)
    amax = np.abs(x).reshape(64, 8, 32).max(-1)
    assert np.array_equal(sv, 2.0 ** (np.floor(np.log2(amax)) - 2))


def test_mxfp4_scale_range():
    tiny = _bits(np.full((1, 32), 2.0 ** -15, np.float32))      # shared_exp = -17: below the stored range
    c, s = oracle.quantize_variant(tiny, 32, oracle.MXFP4)
    assert s.max() == 0 and np.all(oracle.dequantize(c, s, 32) == 0)
    edge = _bits(np.full((1, 32), 2.0 ** -14, np.float32))      # shared_exp = -16: the smallest subnormal scale
    c, s = oracle.quantize_variant(edge, 32, oracle.MXFP4)
    assert s[0, 0, 0] == 1 and np.all(oracle.dequantize(c, s, 32) == 2.0 ** -14)
    huge = _bits(np.full((1, 32), 2.0 ** 20, np.float32))       # shared_exp = 18 -> stored as 2^15, elements clamp
    c, s = oracle.quantize_variant(huge, 32, oracle.MXFP4)
    assert oracle.e5m2_value(int(s[0, 0, 0])) == 2.0 ** 15 and np.all(oracle.dequantize(c, s, 32) == 6 * 2.0 ** 15)


def test_symmetric_fp8_is_the_one_sided_quantizer_on_magnitudes():
    """One scale from max|x| / 6: magnitudes and scale are those of the (pinned) AMXFP4 quantizer applied to |x|,
    whose positive side then holds every element; the sign bits are the input's."""
    for kind in ("normal", "mixed", "wide"):
        bits = inputs.random_groups(33, 48, 256, kind)
        c, s = oracle.quantize_variant(bits, 32, oracle.SYMMETRIC_FP8)
        ca, sa = oracle.quantize(bits & 0x7FFF, 32)
        assert np.array_equal(s[..., 0], sa[..., 0]) and np.array_equal(s[..., 1], sa[..., 0])
        c4, ca4 = oracle.unpack_codes(c), oracle.unpack_codes(ca)
        assert np.array_equal(c4 & 7, ca4 & 7)
        assert np.array_equal(c4 >> 3, (bits >> 15).astype(np.uint8))
    # negating the input flips sign bits only
    c2, s2 = oracle.quantize_variant(bits ^ 0x8000, 32, oracle.SYMMETRIC_FP8)
    assert np.array_equal(s2, s) and np.array_equal(oracle.unpack_codes(c2), oracle.unpack_codes(c) ^ 8)


def test_symmetric_formats_lose_to_amxfp4_on_skewed_groups():
    """Section 4.3's point, as an invariant: with one scale per group the smaller side of a skewed group is
    quantized with the larger side's scale; the asymmetric format's error is never larger on such data."""
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.uniform(0, 31, (64, 16)), -rng.uniform(0, 4.9, (64, 16))], axis=1).astype(np.float32)
    bits = _bits(x)
    xr = inputs.bf16_bits_to_f32(bits).astype(np.float64)
    err = {}
    for name, (c, s) in {"amx": oracle.quantize(bits, 32), "sym": oracle.quantize_variant(bits, 32, oracle.SYMMETRIC_FP8),
                         "mx": oracle.quantize_variant(bits, 32, oracle.MXFP4)}.items():
        err[name] = np.mean((oracle.dequantize(c, s, 32) - xr) ** 2)
    assert err["amx"] < err["sym"] < err["mx"]


def test_per_sign_power_of_two_reproduces_the_printed_value_set():
    """Appendix B.3 prints the values of "AMXFP4 (Shared Scale: PoT)" on linspace(-4.9, 31, 1024) as one group."""
    path = os.path.join(os.path.dirname(__file__), "golden", "worked_example.txt")
    printed = next(line.split()[1:] for line in open(path) if line.startswith("amxfp4_pot "))
    x = _bits(np.linspace(-4.9, 31, 1024, dtype=np.float32))[None, :]
    c, s = oracle.quantize_variant(x, 1024, oracle.AMXFP4_POT)
    assert np.unique(oracle.dequantize(c, s, 1024)).tolist() == sorted(float(t) for t in printed)
    assert oracle.e5m2_value(int(s[0, 0, 0])) == 4.0 and oracle.e5m2_value(int(s[0, 0, 1])) == 1.0


def test_per_sign_power_of_two_equals_algorithm1_per_sign():
    bits = inputs.random_groups(35, 64, 256, "normal")
    x = inputs.bf16_bits_to_f32(bits).astype(np.float64)
    c, s = oracle.quantize_variant(bits, 32, oracle.AMXFP4_POT)
    assert np.array_equal(oracle.dequantize(c, s, 32), oracle.fakequant_pot_floor(x, 32, asym=True))


def test_power_of_two_round_scale():
    """Exponent rounded instead of floored: the scale is 2^(round(log2 max) - 2) (numpy's log2 as the independent
    route; a tie would need max = sqrt(2) * 2^e, which no bf16 value is), so max / scale lies in [2^1.5, 2^2.5) and
    never reaches past 6: the clamping error the appendix attributes to the floor is gone.  Elements are rounded as
    in every other format (checked against the pinned one-scale quantizer run with that scale's group maximum)."""
    for mode, per_sign in ((oracle.MXFP4_POT_ROUND, False), (oracle.AMXFP4_POT_ROUND, True)):
        bits = inputs.random_groups(36, 64, 256, "normal")
        x = inputs.bf16_bits_to_f32(bits).astype(np.float64).reshape(64, 8, 32)
        c, s = oracle.quantize_variant(bits, 32, mode)
        sv = s.view(ml_dtypes.float8_e5m2).astype(np.float64)
        pmax, nmax = np.where(x > 0, x, 0).max(-1), np.where(x < 0, -x, 0).max(-1)
        tops = (pmax, nmax) if per_sign else (np.maximum(pmax, nmax),) * 2
        for side, top in enumerate(tops):
            ok = top > 0
            assert np.array_equal(sv[..., side][ok], 2.0 ** (np.rint(np.log2(top[ok])) - 2))
            ratio = top[ok] / sv[..., side][ok]
            assert np.all(ratio >= 2 ** 1.5) and np.all(ratio < 2 ** 2.5)
        assert oracle.quant_error(bits, c, s, 32)[3] == 0
        # floor and round differ exactly where the maximum's mantissa is at least sqrt(2)
        cf, sf = oracle.quantize_variant(bits, 32, oracle.AMXFP4_POT if per_sign else oracle.MXFP4)
        svf = sf.view(ml_dtypes.float8_e5m2).astype(np.float64)
        for side, top in enumerate(tops):
            ok = top > 0
            up = top[ok] / 2.0 ** np.floor(np.log2(top[ok])) >= np.sqrt(2.0)
            assert np.array_equal(sv[..., side][ok] / svf[..., side][ok], np.where(up, 2.0, 1.0))
        # element codes: a group whose scale did not move has the floor variant's codes
        same = np.all(sv == svf, axis=-1)
        c4, cf4 = oracle.unpack_codes(c).reshape(64, 8, 32), oracle.unpack_codes(cf).reshape(64, 8, 32)
        assert np.array_equal(c4[same], cf4[same]) and same.any() and (~same).any()
