"""Pins for the oracle's quantization-error split (max-clamping vs. rounding error, appendix "Determining PoT Shared
Scale: Floor vs. Round"): the numbers the worked example of Appendix B.3 prints, hand-worked groups, and invariants."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2411_09909_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "quant_error_cases.txt")
FORMATS = {"amxfp4": None, "sym_fp8": oracle.SYMMETRIC_FP8, "mxfp4": oracle.MXFP4}


def _quantize(bits, gs, fmt):
    return oracle.quantize(bits, gs) if FORMATS[fmt] is None else oracle.quantize_variant(bits, gs, FORMATS[fmt])


def test_worked_example_clamping():
    """Appendix B.3: with the FP8 scale 31 is represented by 30 and -4.9 by -5.25; with the power-of-two scale the
    largest value is 24.  So the clamped elements are exactly those above 30 (resp. 24), each with error x - 30
    (x - 24), and the negative side clamps nothing."""
    x = torch.linspace(-4.9, 31, 1024).to(torch.bfloat16)
    bits = x.view(torch.int16).numpy().view(np.uint16)[None, :]
    xv = x.double().numpy()
    for fmt, top in (("amxfp4", 30.0), ("mxfp4", 24.0)):
        e = oracle.quant_error(bits, *_quantize(bits, 1024, fmt), 1024)
        over = xv[xv > top]
        assert e[3] == len(over) > 0
        assert e[2] == pytest.approx(np.sum((over - top) ** 2), rel=1e-13)
        assert e[0] == pytest.approx(np.sum(xv ** 2), rel=1e-13)
        assert e[1] > e[2]


def test_hand_worked_groups():
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        name, fmt, vals, total, clamped, count = [t.strip() for t in line.split("|")]
        x = np.zeros((1, 16), np.float32)
        v = [float(t) for t in vals.split()]
        x[0, :len(v)] = v
        bits = inputs.f32_to_bf16_bits(x)
        e = oracle.quant_error(bits, *_quantize(bits, 16, fmt), 16)
        assert (e[1], e[2], e[3]) == (float(total), float(clamped), float(count)), name


@pytest.mark.parametrize("fmt", list(FORMATS))
@pytest.mark.parametrize("gs", [16, 32, 128])
def test_invariants(fmt, gs):
    bits = inputs.random_groups(77 + gs, 8, 512, "normal")
    q = _quantize(bits, gs, fmt)
    e = oracle.quant_error(bits, *q, gs)
    x = inputs.bf16_bits_to_f32(bits).astype(np.float64)
    # total error is the distance to the decoded tensor; the clamped part never exceeds it
    assert e[1] == pytest.approx(np.sum((x - oracle.dequantize(*q, gs)) ** 2), rel=1e-12)
    assert 0 <= e[2] <= e[1] and e[0] == pytest.approx(np.sum(x * x), rel=1e-12)
    # multiplying the input by 4 multiplies scales by 4 and every error by 16; codes do not change
    bits4 = inputs.f32_to_bf16_bits((x * 4).astype(np.float32))
    q4 = _quantize(bits4, gs, fmt)
    assert np.array_equal(q4[0], q[0])
    e4 = oracle.quant_error(bits4, *q4, gs)
    assert np.allclose(e4[:3], 16 * e[:3], rtol=1e-12) and e4[3] == e[3]
    # a decoded tensor is represented exactly: quantizing it again leaves no error
    xh = oracle.dequantize(*q, gs)
    if np.all(np.abs(xh) < 3e38):
        bh = inputs.f32_to_bf16_bits(xh.astype(np.float32))
        assert np.array_equal(inputs.bf16_bits_to_f32(bh).astype(np.float64), xh)
        # same scales are re-derived only when a side's extreme sits on +-6: check the weaker, always-true fact
        assert oracle.quant_error(bh, *q, gs)[1] == 0.0


def test_fp8_scale_clamps_less_than_power_of_two_floor():
    """Direction of the appendix's finding: under the floor power-of-two scale max / scale reaches up to 8, under the
    nearest-FP8 scale it stays within [5.4, 6.75]: about as many elements are clamped (a scale rounded down clamps
    its maximum), but by much less."""
    bits = inputs.activation(2, 0, M=64)
    e_fp8 = oracle.quant_error(bits, *_quantize(bits, 32, "sym_fp8"), 32)
    e_pot = oracle.quant_error(bits, *_quantize(bits, 32, "mxfp4"), 32)
    assert e_pot[2] > 3 * e_fp8[2] and e_pot[3] > 0 and e_fp8[3] > 0
