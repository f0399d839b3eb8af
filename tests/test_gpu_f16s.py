"""GPU parity of FP4 with binary16 shared scales (the FP16 row of the appendix's scale-encoding ablation): codes and
scale patterns bit for bit against the CPU oracle, decoded values exactly, the product within 1e-5 relative Frobenius
error (fp32 accumulation against the oracle's fp64), the error sums within 2^-20 with an exact clamped count."""
import numpy as np
import pytest
import torch

import oracle
from paper_2411_09909_b200 import amx, inputs

pytestmark = pytest.mark.gpu


def dev_bf16(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def host_u16(t):
    return t.cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("asym", [False, True])
@pytest.mark.parametrize("gs", [16, 32, 64, 128])
@pytest.mark.parametrize("kind,rows,K", [("normal", 257, 1280), ("mixed", 96, 512), ("wide", 40, 256), ("normal", 1, 128)])
def test_quantize_f16s_bit_exact(asym, gs, kind, rows, K):
    bits = inputs.random_groups(3100 + rows + gs, rows, K, kind)
    wide = torch.zeros((rows, K + 72), dtype=torch.bfloat16, device="cuda")
    wide[:, 8:8 + K] = dev_bf16(bits)
    oc, os_ = oracle.quantize_f16s(bits, gs, asym)
    for x in (dev_bf16(bits), wide[:, 8:8 + K]):                       # contiguous and row-strided input
        c, s = amx.quantize_f16s(x, gs, asym)
        assert np.array_equal(host_u16(s), os_)
        assert np.array_equal(c.cpu().numpy(), oc)
    d = amx.dequantize_f16s(c, s, gs).cpu().numpy()
    assert np.array_equal(d, oracle.dequantize_f16s(oc, os_, gs).astype(np.float32))
    assert np.array_equal(d.astype(np.float64), oracle.dequantize_f16s(oc, os_, gs))     # exact in fp32


@pytest.mark.parametrize("asym", [False, True])
@pytest.mark.parametrize("gs", [16, 128])
def test_quantize_e4m3_scale_bit_exact(asym, gs):
    for kind, rows, K in (("normal", 130, 768), ("mixed", 64, 512), ("wide", 40, 256)):
        bits = inputs.random_groups(3600 + rows + gs, rows, K, kind)
        c, s = amx.quantize_f16s(dev_bf16(bits), gs, asym, e4m3=True)
        oc, os_ = oracle.quantize_f16s(bits, gs, asym, e4m3=True)
        assert np.array_equal(host_u16(s), os_) and np.array_equal(c.cpu().numpy(), oc)
        d = amx.dequantize_f16s(c, s, gs).cpu().numpy()
        assert np.array_equal(d.astype(np.float64), oracle.dequantize_f16s(oc, os_, gs))
    # every bf16 magnitude as a side maximum: E4M3 rounding, subnormals, saturation at 448
    mags = np.arange(0x0001, 0x7F80, dtype=np.uint16)
    n = (mags.size // 64) * 64
    b = np.zeros((n, 16), np.uint16)
    b[:, 2] = mags[:n]
    b[:, 11] = mags[:n][::-1] | 0x8000
    b = b.reshape(-1, 64 * 16)
    c, s = amx.quantize_f16s(dev_bf16(b), 16, asym, e4m3=True)
    oc, os_ = oracle.quantize_f16s(b, 16, asym, e4m3=True)
    assert np.array_equal(host_u16(s), os_) and np.array_equal(c.cpu().numpy(), oc)


def test_every_bf16_value_as_group_maximum_and_as_element():
    """Every finite bf16 magnitude as a side maximum (scale rounding, binary16 subnormals, saturation), and every
    finite bf16 value as an element under a few hundred scales (element rounding and ties)."""
    mags = np.arange(0x0001, 0x7F80, dtype=np.uint16)
    n = (mags.size // 64) * 64
    bits = np.zeros((n, 16), np.uint16)
    bits[:, 5] = mags[:n]
    bits[:, 9] = mags[:n][::-1] | 0x8000
    bits = bits.reshape(-1, 64 * 16)
    for asym in (False, True):
        c, s = amx.quantize_f16s(dev_bf16(bits), 16, asym)
        oc, os_ = oracle.quantize_f16s(bits, 16, asym)
        assert np.array_equal(host_u16(s), os_) and np.array_equal(c.cpu().numpy(), oc)
    # elements: each row holds one maximum (first element of each 32-group) and 31 arbitrary smaller-or-larger values
    rng = np.random.Generator(np.random.Philox(24110977))
    allv = np.concatenate([np.arange(0x0000, 0x7F80, dtype=np.uint16), np.arange(0x8000, 0xFF80, dtype=np.uint16)])
    reps = 6
    el = np.tile(allv, reps)
    rng.shuffle(el)
    el = el[: (el.size // 31) * 31].reshape(-1, 31)
    mx = inputs.f32_to_bf16_bits((rng.standard_normal(el.shape[0]) * 2.0 ** rng.integers(-12, 12, el.shape[0])).astype(np.float32))
    g = np.concatenate([mx[:, None], el], axis=1)
    g = g[: (g.shape[0] // 8) * 8].reshape(-1, 8 * 32)
    c, s = amx.quantize_f16s(dev_bf16(g), 32, True)
    oc, os_ = oracle.quantize_f16s(g, 32, True)
    assert np.array_equal(host_u16(s), os_) and np.array_equal(c.cpu().numpy(), oc)


@pytest.mark.parametrize("gs", [16, 32, 128])
@pytest.mark.parametrize("M,N,K", [(70, 130, 384), (1, 64, 128), (129, 65, 1024)])
def test_gemm_f16s(gs, M, N, K):
    a = inputs.random_groups(3300 + M, M, K, "normal")
    w = inputs.random_groups(3400 + N, N, K, "mixed")
    w = np.where((w & 0x7F80) > 0x5000, w & 0x8000, w).astype(np.uint16)      # keep products inside fp32
    ca, sa = amx.quantize_f16s(dev_bf16(a), gs, True)
    cw, sw = amx.quantize_f16s(dev_bf16(w), gs, False)
    got = amx.gemm_f16s(ca, sa, cw, sw, gs).cpu().numpy()
    ref = oracle.gemm_f16s(ca.cpu().numpy(), host_u16(sa), cw.cpu().numpy(), host_u16(sw), gs).astype(np.float64)
    assert np.linalg.norm(got - ref) <= 1e-5 * np.linalg.norm(ref)


def test_gemm_f16s_exact_integers():
    rng = np.random.default_rng(35)
    A = rng.integers(-4, 5, (33, 256)).astype(np.float32)
    W = rng.integers(-4, 5, (47, 256)).astype(np.float32)
    A[A == 5] = 4; W[W == 5] = 4
    A[:, ::16], A[:, 1::16], W[:, ::16], W[:, 1::16] = 6, -6, 6, -6
    ca, sa = amx.quantize_f16s(dev_bf16(inputs.f32_to_bf16_bits(A)), 16, True)
    cw, sw = amx.quantize_f16s(dev_bf16(inputs.f32_to_bf16_bits(W)), 16, True)
    got = amx.gemm_f16s(ca, sa, cw, sw, 16).cpu().numpy()
    assert np.array_equal(got, (A.astype(np.int64) @ W.astype(np.int64).T).astype(np.float32))


@pytest.mark.parametrize("asym", [False, True])
@pytest.mark.parametrize("gs", [16, 128])
def test_quant_error_f16s(asym, gs):
    bits = inputs.activation(2, 0, M=192)[:, :1024].copy()
    c, s = amx.quantize_f16s(dev_bf16(bits), gs, asym)
    got = amx.quant_error_f16s(dev_bf16(bits), c, s, gs).cpu().numpy()
    ref = oracle.quant_error_f16s(bits, c.cpu().numpy(), host_u16(s), gs)
    assert got[3] == ref[3]
    for i in range(3):
        assert abs(got[i] - ref[i]) <= 2.0 ** -20 * abs(ref[i]) + 1e-300
    # a scale one binary16 rounding below max / 6 clamps by at most that rounding: the clamping part is tiny
    assert ref[2] <= 2.0 ** -20 * ref[0]


def test_f16s_argument_errors():
    L = amx.lib()
    x = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    c = torch.zeros((4, 32), dtype=torch.uint8, device="cuda")
    s = torch.zeros((4, 2, 2), dtype=torch.int16, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    assert L.amx_quantize_f16s(x.data_ptr(), 4, 64, 64, 24, 0, c.data_ptr(), s.data_ptr(), st) == -2
    assert L.amx_quantize_f16s(x.data_ptr(), 4, 64, 64, 32, 4, c.data_ptr(), s.data_ptr(), st) == -5
    assert L.amx_quantize_f16s(None, 4, 64, 64, 32, 0, c.data_ptr(), s.data_ptr(), st) == -1
    assert L.amx_quantize_f16s(x.data_ptr() + 2, 4, 64, 64, 32, 0, c.data_ptr(), s.data_ptr(), st) == -3
    assert L.amx_quantize_f16s(x.data_ptr(), 0, 64, 64, 32, 0, None, None, st) == 0
    o = torch.zeros((4, 64), dtype=torch.float32, device="cuda")
    assert L.amx_dequantize_f16s(c.data_ptr(), s.data_ptr(), 4, 64, 32, o.data_ptr(), 32, st) == -2
    assert L.amx_gemm_f16s(c.data_ptr(), s.data_ptr(), c.data_ptr(), s.data_ptr(), 4, 4, 64, 32, None, 4, st) == -1
    torch.cuda.synchronize()
