"""Scales the FP4 tensor-core kernel cannot represent.  Its scale type spans 15 binades per operand row; a nonzero
scale further below the row's largest one is flushed.  The flushed scales are counted, the explicit FP4 kernel's
error on an adversarial (valid) input is recorded, and the default kernel choice must stay exact on it by running
the bf16-decode kernel instead - a decision taken on the device."""
import numpy as np
import pytest
import torch

import oracle
from paper_2411_09909_b200 import amx, inputs

pytestmark = pytest.mark.gpu

M, N, K = 128, 256, 8192


def dev_bf16(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def rel_fro(got, ref):
    return np.linalg.norm(got.astype(np.float64) - ref) / np.linalg.norm(ref)


def adversarial_operands(binades_below):
    """Every row of A: one dominant group (elements 6 * 2^10) and 255 groups whose scale lies `binades_below`
    binades under it, all positive, against an all-positive weight: the small groups' contributions add up
    coherently."""
    a = np.full((M, K), 6.0 * 2.0 ** (10 - binades_below), np.float32)
    a[:, :32] = 6.0 * 2.0 ** 10
    w = np.ones((N, K), np.float32)
    return inputs.f32_to_bf16_bits(a), inputs.f32_to_bf16_bits(w)


def test_flushed_scales_are_counted_and_auto_stays_exact():
    a_bits, w_bits = adversarial_operands(15)
    qa, qw = oracle.quantize(a_bits, 32), oracle.quantize(w_bits, 32)
    ref = oracle.gemm(*qa, *qw, 32)
    dev = [torch.from_numpy(t).cuda() for t in (*qa, *qw)]
    L = amx.lib()
    assert L.amx_gemm_kernel_for(M, N, K, 32, amx.GEMM_AUTO) == amx.GEMM_FP4
    # the FP4 kernel when asked for explicitly: 255 positive-side scales per row of A are flushed, the result is off
    # by their share, 255 * 2^-15 = 0.78 %
    ws = torch.empty(L.amx_workspace_bytes(M, N, K, 32, amx.GEMM_FP4), dtype=torch.uint8, device="cuda")
    got = amx.gemm(*dev, 32, amx.GEMM_FP4, workspace=ws).cpu().numpy()
    assert amx.gemm_status(ws) == 0
    assert amx.gemm_flushed_scales(ws) == M * (K // 32 - 1)
    err = rel_fro(got, ref)
    assert 5e-3 < err < 1e-2, err
    # the default choice notices the flushed scales on the device and computes the product exactly instead
    ws = torch.empty(L.amx_workspace_bytes(M, N, K, 32, amx.GEMM_AUTO), dtype=torch.uint8, device="cuda")
    got = amx.gemm(*dev, 32, amx.GEMM_AUTO, workspace=ws).cpu().numpy()
    assert amx.gemm_status(ws) == 0
    assert amx.gemm_flushed_scales(ws) == M * (K // 32 - 1)
    assert rel_fro(got, ref) <= 1e-5
    # the same through the one-call layer, with the quantized and with the bf16 weight
    for kw in ({"w_codes": dev[2], "w_scales": dev[3]}, {"w_bf16": dev_bf16(w_bits)}):
        flags_ws = amx.WEIGHT_BF16 if "w_bf16" in kw else 0
        ws = torch.empty(L.amx_quant_gemm_workspace_bytes(M, N, K, 32, flags_ws), dtype=torch.uint8, device="cuda")
        got = amx.quant_gemm(dev_bf16(a_bits), group_size=32, workspace=ws, **kw).cpu().numpy()
        assert amx.gemm_flushed_scales(ws) == M * (K // 32 - 1) and amx.gemm_status(ws) == 0
        assert rel_fro(got, ref) <= 1e-5
    # prepared operands carry the count in their row words, from the separate preparation and from the fused cast
    pa = amx.prepare(dev[0], dev[1], False)
    assert amx.prepared_flushed_scales(pa, M, K, False) == M * (K // 32 - 1)
    _, _, pa2 = amx.quantize_prepared(dev_bf16(a_bits), False)
    assert amx.prepared_flushed_scales(pa2, M, K, False) == M * (K // 32 - 1)
    _, _, pw = amx.quantize_prepared(dev_bf16(w_bits), True)
    assert amx.prepared_flushed_scales(pw, N, K, True) == 0


def test_scales_inside_the_range_are_kept_and_the_fp4_kernel_runs():
    """14 binades below the row's largest scale still fits: nothing is flushed, AUTO stays on the FP4 kernel (its
    result equals the explicit FP4 call bit for bit) and is exact up to summation order."""
    a_bits, w_bits = adversarial_operands(14)
    qa, qw = oracle.quantize(a_bits, 32), oracle.quantize(w_bits, 32)
    ref = oracle.gemm(*qa, *qw, 32)
    dev = [torch.from_numpy(t).cuda() for t in (*qa, *qw)]
    L = amx.lib()
    ws = torch.empty(L.amx_workspace_bytes(M, N, K, 32, amx.GEMM_AUTO), dtype=torch.uint8, device="cuda")
    auto = amx.gemm(*dev, 32, amx.GEMM_AUTO, workspace=ws)
    assert amx.gemm_flushed_scales(ws) == 0 and amx.gemm_status(ws) == 0
    assert torch.equal(auto, amx.gemm(*dev, 32, amx.GEMM_FP4))
    assert rel_fro(auto.cpu().numpy(), ref) <= 1e-4


def test_flushed_count_on_fuzz_rows_matches_host_count():
    """Wide-range fuzz rows: the device's count equals a host-side count from the oracle's scale bytes."""
    bits = inputs.random_groups(1500, 300, 1056, "wide")
    oc, os_ = oracle.quantize(bits, 32)
    b = os_.astype(np.int64)
    key = np.where(b >= 4, (b + 8) >> 2, np.array([0, 1, 2, 2])[np.minimum(b, 3)])      # exponent key of an E5M2 byte
    kmax = key.reshape(300, -1).max(axis=1)
    want = int(np.sum((b != 0) & (kmax[:, None, None] - key >= 15)))
    assert want > 0
    pa = amx.prepare(torch.from_numpy(oc).cuda(), torch.from_numpy(os_).cuda(), False)
    assert amx.prepared_flushed_scales(pa, 300, 1056, False) == want
    _, _, pa2 = amx.quantize_prepared(dev_bf16(bits), False)
    assert amx.prepared_flushed_scales(pa2, 300, 1056, False) == want
