"""GPU parity of NVFP4 / ANVFP4 (group 16, E4M3 group scales, one fp32 tensor scale - the format Section 5 of the
paper compares AMXFP4 with): codes, scale bytes and the tensor scale bit for bit against the CPU oracle, the decoded
values exactly, the product on the FP4 tensor-core kernel within 1e-3 relative Frobenius error of the oracle's."""
import numpy as np
import pytest
import torch

import oracle
from paper_2411_09909_b200 import amx, inputs

pytestmark = pytest.mark.gpu


def dev_bf16(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def rel_fro(got, ref):
    return np.linalg.norm(got.astype(np.float64) - ref) / np.linalg.norm(ref)


@pytest.mark.parametrize("asym", [False, True])
@pytest.mark.parametrize("kind,rows,K", [("normal", 257, 1280), ("mixed", 96, 512), ("wide", 40, 256), ("normal", 1, 64)])
def test_quantize_nvfp4_bit_exact(asym, kind, rows, K):
    bits = inputs.random_groups(2400 + rows, rows, K, kind)
    finite = (bits & 0x7F80) != 0x7F80
    assert finite.all()
    wide = torch.zeros((rows, K + 72), dtype=torch.bfloat16, device="cuda")
    wide[:, 8:8 + K] = dev_bf16(bits)
    for x in (dev_bf16(bits), wide[:, 8:8 + K]):                       # contiguous and row-strided input
        c, s, ts = amx.quantize_nvfp4(x, asym)
        oc, os_, ot = oracle.quantize_nv(bits, asym)
        t = ts.cpu().numpy()
        assert t[0] == ot and t[1] == np.abs(inputs.bf16_bits_to_f32(bits)).max()
        assert np.array_equal(s.cpu().numpy(), os_)
        assert np.array_equal(c.cpu().numpy(), oc)
    d = amx.dequantize_nvfp4(c, s, ts).cpu().numpy()
    assert np.array_equal(d, oracle.dequantize_nv(oc, os_, ot).astype(np.float32))
    db = amx.dequantize_nvfp4(c, s, ts, torch.bfloat16).view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(db, inputs.f32_to_bf16_bits(d))


def test_quantize_nvfp4_all_zero_tensor_and_every_maximum():
    z = torch.zeros((4, 128), dtype=torch.bfloat16, device="cuda")
    c, s, ts = amx.quantize_nvfp4(z, True)
    assert ts.cpu().tolist() == [1.0, 0.0] and not c.any() and not s.any()
    # every positive bf16 value up to the tensor maximum as a group maximum, on both sides
    vals = np.arange(0x0080, 0x4700, dtype=np.uint16)                     # normal bf16 values up to 32768
    bits = np.zeros((vals.size, 16), np.uint16)
    bits[:, 3] = vals
    bits[:, 7] = vals[::-1] | 0x8000
    bits = bits.reshape(-1, 64 * 16)[: (vals.size * 16) // 1024]
    for asym in (False, True):
        c, s, ts = amx.quantize_nvfp4(dev_bf16(bits), asym)
        oc, os_, ot = oracle.quantize_nv(bits, asym)
        assert ts.cpu().numpy()[0] == ot
        assert np.array_equal(s.cpu().numpy(), os_) and np.array_equal(c.cpu().numpy(), oc)


@pytest.mark.parametrize("asym_a,asym_w", [(False, False), (True, True), (True, False)])
@pytest.mark.parametrize("M,N,K", [(300, 520, 1088), (128, 256, 64), (1, 1, 64)])
def test_gemm_nvfp4_against_oracle(asym_a, asym_w, M, N, K):
    a_bits = inputs.random_groups(2500 + M, M, K, "normal")
    w_bits = inputs.random_groups(2501 + N, N, K, "normal")
    qa, qw = oracle.quantize_nv(a_bits, asym_a), oracle.quantize_nv(w_bits, asym_w)
    ref = oracle.gemm_nv(*qa, *qw)
    ca, sa, ta, pa = amx.quantize_nvfp4(dev_bf16(a_bits), asym_a, prepared_as="a")
    cw, sw, tw, pw = amx.quantize_nvfp4(dev_bf16(w_bits), asym_w, prepared_as="w")
    assert np.array_equal(ca.cpu().numpy(), qa[0]) and np.array_equal(cw.cpu().numpy(), qw[0])
    work = torch.full((256,), 0xFF, dtype=torch.uint8, device="cuda")
    got = amx.gemm_nvfp4(pa, pw, M, N, K, workspace=work).cpu().numpy()
    assert amx.gemm_status(work) == 0
    assert rel_fro(got, ref) <= 1e-3
    assert rel_fro(got, ref) <= 1e-5                                      # fp32 accumulation of short products


def test_gemm_nvfp4_full_size_layer_sampled():
    """Config 2's first layer (2048 x 4096 -> 12288) in NVFP4 and ANVFP4, 64 sampled rows against the oracle."""
    a_bits, w_bits = inputs.activation(2, 0), inputs.weight(2, 0)
    M, K, N = 2048, 4096, 12288
    rows = np.sort(np.random.default_rng(26).choice(M, size=64, replace=False))
    for asym in (False, True):
        ca, sa, ta, pa = amx.quantize_nvfp4(dev_bf16(a_bits), asym, prepared_as="a")
        cw, sw, tw, pw = amx.quantize_nvfp4(dev_bf16(w_bits), asym, prepared_as="w")
        oa = oracle.quantize_nv(a_bits, asym)
        assert np.array_equal(ca.cpu().numpy(), oa[0]) and np.array_equal(sa.cpu().numpy(), oa[1]) and ta.cpu().numpy()[0] == oa[2]
        got = amx.gemm_nvfp4(pa, pw, M, N, K)[torch.from_numpy(rows).cuda()].cpu().numpy()
        ref = oracle.gemm_nv(*oa, cw.cpu().numpy(), sw.cpu().numpy(), tw.cpu().numpy()[0], rows=rows)
        assert rel_fro(got, ref) <= 1e-3
