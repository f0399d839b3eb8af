"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Codes and scales must match bit for bit; GEMM outputs within 1e-3 relative Frobenius
error of the oracle's fp64 product of the decoded operands."""
import numpy as np
import pytest
import torch

import oracle
from paper_2411_09909_b200 import amx, inputs

pytestmark = pytest.mark.gpu
GEMM_TOL = 1e-3


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def rel_fro(got: np.ndarray, ref: np.ndarray) -> float:
    den = np.linalg.norm(ref.astype(np.float64))
    num = np.linalg.norm(got.astype(np.float64) - ref.astype(np.float64))
    return num / den if den > 0 else num


def check_quantize(bits, gs=32):
    c, s = amx.quantize(dev_bf16(bits), gs)
    oc, os_ = oracle.quantize(bits, gs)
    assert np.array_equal(c.cpu().numpy(), oc)
    assert np.array_equal(s.cpu().numpy(), os_)
    return c, s


# ------------------------------------------------------------------ quantize --

@pytest.mark.parametrize("gs", [16, 32, 64, 128])
@pytest.mark.parametrize("kind", ["normal", "wide", "mixed"])
def test_quantize_bit_exact_random_groups(gs, kind):
    check_quantize(inputs.random_groups(31, 257, 1280, kind), gs)      # ragged: 257 rows, 10 tiles + tail


def test_quantize_exhaustive_bf16_times_scale_codes():
    """Every finite bf16 value against every normal/subnormal E5M2 scale code, on both sides."""
    finite = np.concatenate([np.arange(0, 0x7F80), np.arange(0x8000, 0xFF80)]).astype(np.uint16)
    per = 30
    n_groups = -(-finite.size // per)
    payload = np.zeros(n_groups * per, np.uint16)
    payload[: finite.size] = finite
    payload = payload.reshape(n_groups, per)
    rows = []
    for sc in range(1, 0x7C):
        m_pos = inputs.f32_to_bf16_bits(np.array([6.0 * oracle.e5m2_value(sc)], np.float32))[0]
        sc_n = (sc * 7) % 0x7B + 1
        m_neg = inputs.f32_to_bf16_bits(np.array([-6.0 * oracle.e5m2_value(sc_n)], np.float32))[0]
        g = np.empty((n_groups, 32), np.uint16)
        g[:, 0], g[:, 1], g[:, 2:] = m_pos, m_neg, payload
        rows.append(g.reshape(-1))
    check_quantize(np.stack(rows), 32)


def test_quantize_scale_rounding_all_maxima():
    """Every finite positive bf16 value as the group maximum (scale = nearest E5M2 of max/6)."""
    vals = np.arange(0, 0x7F80, dtype=np.uint16)
    bits = np.zeros((vals.size, 32), np.uint16)
    bits[:, 5] = vals
    bits[:, 9] = vals[::-1] | 0x8000
    check_quantize(bits.reshape(-1, 32 * 64), 32)


def test_quantize_strided_rows_and_tiny_shapes():
    bits = inputs.random_groups(32, 5, 96, "mixed")
    x = torch.zeros((5, 160), dtype=torch.bfloat16, device="cuda")
    x[:, :96] = dev_bf16(bits)
    c, s = amx.quantize(x[:, :96], 32)
    oc, os_ = oracle.quantize(bits, 32)
    assert np.array_equal(c.cpu().numpy(), oc) and np.array_equal(s.cpu().numpy(), os_)
    check_quantize(inputs.random_groups(33, 1, 32, "normal"), 32)        # a single group
    c0, s0 = amx.quantize(torch.empty((0, 64), dtype=torch.bfloat16, device="cuda"), 32)
    assert c0.shape == (0, 32) and s0.shape == (0, 2, 2)


@pytest.mark.parametrize("gs", [16, 32, 64])
def test_quantize_t_matches_oracle_on_transpose(gs):
    bits = inputs.random_groups(34, 192, 128, "mixed")[:, :100]           # R=192, C=100 (ragged tiles)
    bits = np.ascontiguousarray(bits)
    c, s = amx.quantize_t(dev_bf16(bits), gs)
    oc, os_ = oracle.quantize(np.ascontiguousarray(bits.T), gs)
    assert np.array_equal(c.cpu().numpy(), oc) and np.array_equal(s.cpu().numpy(), os_)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_dequantize_exact(dtype):
    bits = inputs.random_groups(35, 100, 640, "wide")
    oc, os_ = oracle.quantize(bits, 32)
    out = amx.dequantize(torch.from_numpy(oc).cuda(), torch.from_numpy(os_).cuda(), 32, dtype)
    assert np.array_equal(out.double().cpu().numpy(), oracle.dequantize(oc, os_, 32))


def test_dequantize_all_codes_all_scales():
    codes = np.tile(np.arange(16, dtype=np.uint8), 2)                     # one group: every code twice
    packed = oracle.pack_codes(np.tile(codes, (0x7C, 1)))
    scales = np.zeros((0x7C, 1, 2), np.uint8)
    scales[:, 0, 0] = np.arange(0x7C)
    scales[:, 0, 1] = np.arange(0x7C)[::-1]
    out = amx.dequantize(torch.from_numpy(packed).cuda(), torch.from_numpy(scales).cuda(), 32, torch.float32)
    assert np.array_equal(out.double().cpu().numpy(), oracle.dequantize(packed, scales, 32))


# ---------------------------------------------------------------------- GEMM --

def _gemm_case(seed, M, N, K, gs, flags, kind="mixed"):
    a = inputs.random_groups(seed, M, K, kind)
    w = inputs.random_groups(seed + 1, N, K, "normal")
    (ac, as_), (wc, ws) = oracle.quantize(a, gs), oracle.quantize(w, gs)
    got = amx.gemm(*(torch.from_numpy(t).cuda() for t in (ac, as_, wc, ws)), gs, flags).cpu().numpy()
    ref = oracle.gemm(ac, as_, wc, ws, gs)
    return got, ref


@pytest.mark.parametrize("shape", [(1, 1, 32), (70, 130, 96), (128, 256, 512), (200, 72, 1024)])
@pytest.mark.parametrize("gs", [16, 32, 128])
def test_gemm_simt_against_oracle(shape, gs):
    M, N, K = shape
    if K % gs:
        pytest.skip("K not a multiple of the group size")
    got, ref = _gemm_case(41, M, N, K, gs, amx.GEMM_SIMT, "normal")
    assert rel_fro(got, ref) <= GEMM_TOL
    assert rel_fro(got, ref) <= 1e-5          # fp32 accumulation of <= 10-bit products is far tighter


TC_KERNELS = [("tc", 0x20, 1e-5), ("fp4", 0x40, 1e-4)]


@pytest.mark.parametrize("shape", [(128, 256, 64), (128, 256, 256), (1, 1, 32), (130, 260, 96), (300, 520, 1056),
                                   (256, 512, 4096)])
@pytest.mark.parametrize("kernel", TC_KERNELS, ids=lambda k: k[0])
def test_gemm_tensor_core_against_oracle(shape, kernel):
    """tcgen05 paths: one tile, several K blocks, a single group, ragged M/N/K tails, several tiles.
    The bf16-decode kernel is exact up to summation order; the FP4 kernel additionally flushes scales
    more than 14 binades below their row's largest scale."""
    M, N, K = shape
    _, flag, tol = kernel
    assert amx.lib().amx_gemm_kernel_for(M, N, K, 32, flag) == flag
    a = inputs.random_groups(51, M, K, "mixed")
    w = inputs.random_groups(52, N, K, "normal")
    (ac, as_), (wc, ws) = oracle.quantize(a, 32), oracle.quantize(w, 32)
    work = torch.zeros(max(256, amx.lib().amx_workspace_bytes(M, N, K, 32, flag)), dtype=torch.uint8, device="cuda")
    got = amx.gemm(*(torch.from_numpy(t).cuda() for t in (ac, as_, wc, ws)), 32, flag, workspace=work)
    assert amx.gemm_status(work) == 0
    got = got.cpu().numpy()
    ref = oracle.gemm(ac, as_, wc, ws, 32)
    for m in range(M):                         # row-wise: "mixed" rows differ by many orders of magnitude
        if np.all(np.isfinite(ref[m])) and np.linalg.norm(ref[m]) > 0:
            assert rel_fro(got[m], ref[m]) <= tol, m


@pytest.mark.parametrize("kernel", TC_KERNELS, ids=lambda k: k[0])
def test_gemm_tensor_core_exact_on_small_integers(kernel):
    rng = np.random.default_rng(9)
    grid = np.array([0, 1, 2, 3, 4, 6], np.float32)
    def ints(r, k):
        t = grid[rng.integers(0, 6, size=(r, k))] * rng.choice([-1.0, 1.0], size=(r, k)).astype(np.float32)
        t[:, ::32], t[:, 1::32] = 6.0, -6.0
        return t
    a, w = ints(200, 320), ints(300, 320)
    qa, qw = oracle.quantize(inputs.f32_to_bf16_bits(a), 32), oracle.quantize(inputs.f32_to_bf16_bits(w), 32)
    got = amx.gemm(*(torch.from_numpy(t).cuda() for t in (*qa, *qw)), 32, kernel[1]).cpu().numpy()
    assert np.array_equal(got, (a.astype(np.int64) @ w.astype(np.int64).T).astype(np.float32))


def test_gemm_fp4_scale_range_handling():
    """Rows whose scales span more than the UE4M3 range: the small groups are flushed, the result stays
    within 2^-13 of the row's norm; rows of zeros and one-sided rows give exact zeros / exact values."""
    rng = np.random.default_rng(10)
    a = rng.standard_normal((64, 256)).astype(np.float32)
    a[:, 32:64] *= 2.0 ** 20                    # one dominant group per row, 20 binades above the rest
    a[5] = 0.0                                  # all-zero row
    a[6] = np.abs(a[6])                         # no negative side
    w = rng.standard_normal((96, 256)).astype(np.float32)
    w[:, :32] *= 2.0 ** -18
    qa, qw = oracle.quantize(inputs.f32_to_bf16_bits(a), 32), oracle.quantize(inputs.f32_to_bf16_bits(w), 32)
    got = amx.gemm(*(torch.from_numpy(t).cuda() for t in (*qa, *qw)), 32, amx.GEMM_FP4).cpu().numpy()
    ref = oracle.gemm(*qa, *qw, 32)
    assert np.all(got[5] == 0.0)
    for m in range(64):
        if m != 5:
            assert rel_fro(got[m], ref[m]) <= 2.0 ** -13


@pytest.mark.parametrize("flag", [0x20, 0x40], ids=["tc", "fp4"])
def test_gemm_tensor_core_matches_simt_at_scale(flag):
    a = dev_bf16(inputs.activation(2, 1))                 # 2048 x 4096
    w = dev_bf16(inputs.weight(2, 1))                     # 4096 x 4096
    (ac, as_), (wc, ws) = amx.quantize(a, 32), amx.quantize(w, 32)
    tc = amx.gemm(ac, as_, wc, ws, 32, flag)
    simt = amx.gemm(ac, as_, wc, ws, 32, amx.GEMM_SIMT)
    assert rel_fro(tc.cpu().numpy(), simt.cpu().numpy()) <= 1e-5


def test_gemm_prepared_two_phase_equals_one_call():
    a = inputs.random_groups(61, 300, 1056, "mixed")
    w = inputs.random_groups(62, 520, 1056, "normal")
    (ac, as_), (wc, ws) = oracle.quantize(a, 32), oracle.quantize(w, 32)
    ac, as_, wc, ws = (torch.from_numpy(t).cuda() for t in (ac, as_, wc, ws))
    pa, pw = amx.prepare(ac, as_, False), amx.prepare(wc, ws, True)
    one = amx.gemm(ac, as_, wc, ws, 32, amx.GEMM_FP4)
    for _ in range(2):                                       # the prepared weight is reused
        assert torch.equal(amx.gemm_prepared(pa, pw, 300, 520, 1056), one)


@pytest.mark.parametrize("a_side,w_side", [(1, 0), (0, -1), (1, 1), (-1, 1), (2, 0)])
def test_gemm_fp4_one_sided_operands(a_side, w_side):
    """Operands without negative (or without positive) elements have an all-zero sign plane; the FP4 kernel then
    does not issue that plane's products.  side: 0 = mixed signs, +1 / -1 = all elements of that sign,
    2 = the first 128 rows non-negative and the rest mixed (tiles differ)."""
    def one_sided(bits, side):
        x = bits.copy()
        if side == 1:
            x &= 0x7FFF
        elif side == -1:
            x |= 0x8000
        elif side == 2:
            x[:128] &= 0x7FFF
        return x
    a = one_sided(inputs.random_groups(71, 300, 1056, "normal"), a_side)
    w = one_sided(inputs.random_groups(72, 520, 1056, "normal"), w_side)
    qa, qw = oracle.quantize(a, 32), oracle.quantize(w, 32)
    ref = oracle.gemm(*qa, *qw, 32)
    dev = [torch.from_numpy(t).cuda() for t in (*qa, *qw)]
    assert rel_fro(amx.gemm(*dev, 32, amx.GEMM_FP4).cpu().numpy(), ref) <= GEMM_TOL
    # through the fused cast as well
    _, _, pa = amx.quantize_prepared(dev_bf16(a), False)
    _, _, pw = amx.quantize_prepared(dev_bf16(w), True)
    assert rel_fro(amx.gemm_prepared(pa, pw, 300, 520, 1056).cpu().numpy(), ref) <= GEMM_TOL


@pytest.mark.parametrize("fmt,mode", [(amx.FMT_SYM_FP8, oracle.SYMMETRIC_FP8), (amx.FMT_MXFP4, oracle.MXFP4)])
def test_symmetric_formats(fmt, mode):
    """The paper's symmetric comparison formats: codes and scales bit-exact against the oracle for every group
    size, on fuzz rows (ties, tiny, huge, one-sided and all-zero groups); the GEMMs take them unchanged; the FP4
    kernel needs one product per tile pair for them, from the fused cast and from amx_prepare alike."""
    for gs in (16, 32, 64, 128):
        for kind in ("mixed", "wide"):
            bits = inputs.random_groups(300 + gs, 96, 512, kind)
            c, s_ = amx.quantize(dev_bf16(bits), gs, fmt=fmt)
            oc, os_ = oracle.quantize_variant(bits, gs, mode)
            assert np.array_equal(c.cpu().numpy(), oc) and np.array_equal(s_.cpu().numpy(), os_), (gs, kind)
    # every bf16 value as a group maximum, and every bf16 value against a fixed maximum
    allv = np.arange(0x7F80, dtype=np.uint16)
    bits = np.zeros((allv.size, 32), np.uint16)
    bits[:, 0] = allv
    bits[:, 1] = allv | 0x8000
    bits[:, 2] = 0x3F80
    c, s_ = amx.quantize(dev_bf16(bits), 32, fmt=fmt)
    oc, os_ = oracle.quantize_variant(bits, 32, mode)
    assert np.array_equal(c.cpu().numpy(), oc) and np.array_equal(s_.cpu().numpy(), os_)
    bits = np.full((allv.size, 32), 0x0000, np.uint16)
    bits[:, 0] = 0x4416                                     # 600.0: the scale is fixed, every value is an element
    bits[:, 1] = allv
    bits[:, 2] = allv | 0x8000
    c, s_ = amx.quantize(dev_bf16(bits), 32, fmt=fmt)
    oc, os_ = oracle.quantize_variant(bits, 32, mode)
    assert np.array_equal(c.cpu().numpy(), oc) and np.array_equal(s_.cpu().numpy(), os_)
    # products
    a_bits = inputs.random_groups(311, 300, 1056, "normal")
    w_bits = inputs.random_groups(312, 520, 1056, "normal")
    qa, qw = oracle.quantize_variant(a_bits, 32, mode), oracle.quantize_variant(w_bits, 32, mode)
    ref = oracle.gemm(*qa, *qw, 32)
    ac, as_ = amx.quantize(dev_bf16(a_bits), 32, fmt=fmt)
    wc, ws = amx.quantize(dev_bf16(w_bits), 32, fmt=fmt)
    for flags in (amx.GEMM_SIMT, amx.GEMM_TC, amx.GEMM_FP4):
        assert rel_fro(amx.gemm(ac, as_, wc, ws, 32, flags).cpu().numpy(), ref) <= GEMM_TOL, flags
    c2, s2, pa = amx.quantize_prepared(dev_bf16(a_bits), False, fmt=fmt)
    _, _, pw = amx.quantize_prepared(dev_bf16(w_bits), True, fmt=fmt)
    assert torch.equal(c2, ac) and torch.equal(s2, as_)
    got = amx.gemm_prepared(pa, pw, 300, 520, 1056)
    assert rel_fro(got.cpu().numpy(), ref) <= GEMM_TOL
    # a symmetric operand against an asymmetric one
    wq = oracle.quantize(w_bits, 32)
    pw_amx = amx.prepare(*(torch.from_numpy(t).cuda() for t in wq), True)
    assert rel_fro(amx.gemm_prepared(pa, pw_amx, 300, 520, 1056).cpu().numpy(), oracle.gemm(*qa, *wq, 32)) <= GEMM_TOL


@pytest.mark.parametrize("fmt,mode", [(amx.FMT_AMXFP4_POT, oracle.AMXFP4_POT), (amx.FMT_MXFP4_POT_ROUND, oracle.MXFP4_POT_ROUND),
                                      (amx.FMT_AMXFP4_POT_ROUND, oracle.AMXFP4_POT_ROUND)])
def test_power_of_two_scale_formats(fmt, mode):
    """Power-of-two shared scales (per-sign floor; exponent rounded, per group and per sign): codes and scales
    bit-exact against the oracle for every group size, every bf16 value as a side maximum and as an element; the
    GEMMs take the stored operands unchanged."""
    for gs in (16, 32, 64, 128):
        for kind in ("mixed", "wide"):
            bits = inputs.random_groups(340 + gs, 96, 512, kind)
            c, s_ = amx.quantize(dev_bf16(bits), gs, fmt=fmt)
            oc, os_ = oracle.quantize_variant(bits, gs, mode)
            assert np.array_equal(c.cpu().numpy(), oc) and np.array_equal(s_.cpu().numpy(), os_), (gs, kind)
    allv = np.arange(0x7F80, dtype=np.uint16)
    bits = np.zeros((allv.size, 32), np.uint16)
    bits[:, 0] = allv
    bits[:, 1] = allv[::-1] | 0x8000                        # the two sides get different maxima
    bits[:, 2] = 0x3F80
    c, s_ = amx.quantize(dev_bf16(bits), 32, fmt=fmt)
    oc, os_ = oracle.quantize_variant(bits, 32, mode)
    assert np.array_equal(c.cpu().numpy(), oc) and np.array_equal(s_.cpu().numpy(), os_)
    bits = np.full((allv.size, 32), 0x0000, np.uint16)
    bits[:, 0] = 0x4416                                     # 600.0 and -37.0 fix the scales
    bits[:, 3] = 0xC214
    bits[:, 1] = allv
    bits[:, 2] = allv | 0x8000
    c, s_ = amx.quantize(dev_bf16(bits), 32, fmt=fmt)
    oc, os_ = oracle.quantize_variant(bits, 32, mode)
    assert np.array_equal(c.cpu().numpy(), oc) and np.array_equal(s_.cpu().numpy(), os_)
    a_bits = inputs.random_groups(351, 200, 1056, "normal")
    w_bits = inputs.random_groups(352, 264, 1056, "normal")
    qa, qw = oracle.quantize_variant(a_bits, 32, mode), oracle.quantize_variant(w_bits, 32, mode)
    ref = oracle.gemm(*qa, *qw, 32)
    ac, as_ = amx.quantize(dev_bf16(a_bits), 32, fmt=fmt)
    wc, ws = amx.quantize(dev_bf16(w_bits), 32, fmt=fmt)
    for flags in (amx.GEMM_SIMT, amx.GEMM_TC, amx.GEMM_FP4):
        assert rel_fro(amx.gemm(ac, as_, wc, ws, 32, flags).cpu().numpy(), ref) <= GEMM_TOL, flags


@pytest.mark.parametrize("M,N,K", [(1, 12288, 4096), (16, 600, 4096), (130, 300, 2048), (7, 256, 11008)])
def test_gemm_tc_few_tiles_long_k(M, N, K):
    """A few token rows against a big weight (decode-like): the bf16-decode kernel cuts K into slices that run as
    separate CTAs and adds their partial products in slice order; run-to-run identical, padded output untouched,
    and the cast-in-kernel variant takes the same route."""
    a_bits = inputs.random_groups(700 + M, M, K, "normal")
    w_bits = inputs.random_groups(701 + N, N, K, "normal")
    qa, qw = oracle.quantize(a_bits, 32), oracle.quantize(w_bits, 32)
    ref = oracle.gemm(*qa, *qw, 32)
    dev = [torch.from_numpy(t).cuda() for t in (*qa, *qw)]
    assert amx.lib().amx_workspace_bytes(M, N, K, 32, amx.GEMM_TC) > 256          # slices are in use
    wide = torch.full((M, N + 12), 5.0, dtype=torch.float32, device="cuda")
    got = amx.gemm(*dev, 32, amx.GEMM_TC, out=wide[:, :N])
    assert rel_fro(got.cpu().numpy(), ref) <= 1e-5
    assert torch.all(wide[:, N:] == 5.0)
    assert torch.equal(amx.gemm(*dev, 32, amx.GEMM_TC), got.contiguous())
    fused = amx.quant_gemm(dev_bf16(a_bits), dev[2], dev[3], 32, flags=amx.GEMM_TC | amx.GEMM_CAST_IN_KERNEL)
    assert torch.equal(fused, got.contiguous())


@pytest.mark.parametrize("M,N,K", [(16, 1200, 4096), (130, 300, 2048), (1, 256, 11264)])
def test_gemm_prepared_few_tiles_long_k(M, N, K):
    """The FP4 kernel on prepared operands with few output tiles and a long K: with the larger workspace the K
    range is cut into ranges that run as separate work items; partial products are added in range order."""
    a_bits = inputs.random_groups(800 + M, M, K, "normal")
    w_bits = inputs.random_groups(801 + N, N, K, "normal")
    qa, qw = oracle.quantize(a_bits, 32), oracle.quantize(w_bits, 32)
    ref = oracle.gemm(*qa, *qw, 32)
    _, _, pa = amx.quantize_prepared(dev_bf16(a_bits), False)
    _, _, pw = amx.quantize_prepared(dev_bf16(w_bits), True)
    assert amx.lib().amx_gemm_prepared_workspace_bytes(M, N, K, 32) > 256
    wide = torch.full((M, N + 12), 5.0, dtype=torch.float32, device="cuda")
    got = amx.gemm_prepared(pa, pw, M, N, K, out=wide[:, :N])                     # sliced (default workspace)
    assert rel_fro(got.cpu().numpy(), ref) <= 1e-5
    assert torch.all(wide[:, N:] == 5.0)
    assert torch.equal(amx.gemm_prepared(pa, pw, M, N, K), got.contiguous())
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    one = amx.gemm_prepared(pa, pw, M, N, K, workspace=small)                     # 256 bytes: one range
    assert rel_fro(one.cpu().numpy(), ref) <= 1e-5


@pytest.mark.parametrize("M,N,K,kind", [(16, 4096, 4096, "normal"), (1, 12288, 4096, "normal"), (5, 600, 1024, "wide"),
                                        (16, 8, 128, "mixed"), (3, 130, 256, "normal"), (7, 256, 11008, "normal"),
                                        (16, 1030, 11264, "mixed"), (9, 129, 640, "wide"), (17, 300, 1024, "normal"),
                                        (32, 4096, 4096, "normal"), (33, 200, 2304, "mixed"), (64, 1030, 11008, "normal"),
                                        (50, 129, 640, "wide")])
def test_gemm_rows_weight_streaming(M, N, K, kind):
    """At most 64 token rows against a canonical weight (decode phase): the weight-streaming kernel decodes both
    operands exactly, cuts K into ranges over a cluster and adds them in rank order: close to the fp64 oracle,
    run-to-run identical, padded output untouched; AUTO picks it, and amx_quant_gemm (cast of the rows fused with
    their decode) gives the same bits."""
    a_bits = inputs.random_groups(900 + M, M, K, kind)
    w_bits = inputs.random_groups(901 + N, N, K, kind)
    qa, qw = oracle.quantize(a_bits, 32), oracle.quantize(w_bits, 32)
    ref = oracle.gemm(*qa, *qw, 32)
    dev = [torch.from_numpy(t).cuda() for t in (*qa, *qw)]
    assert amx.lib().amx_gemm_kernel_for(M, N, K, 32, amx.GEMM_ROWS) == amx.GEMM_ROWS
    wide = torch.full((M, N + 12), 5.0, dtype=torch.float32, device="cuda")
    got = amx.gemm(*dev, 32, amx.GEMM_ROWS, out=wide[:, :N])
    g = got.cpu().numpy().astype(np.float64)
    if kind == "wide":                           # rows differ by many orders of magnitude: row by row
        for m in range(M):
            if np.all(np.isfinite(ref[m])) and np.linalg.norm(ref[m]) > 0:
                assert rel_fro(g[m], ref[m]) <= 1e-5
    else:
        assert rel_fro(g, ref) <= 1e-5
    assert torch.all(wide[:, N:] == 5.0)
    assert torch.equal(amx.gemm(*dev, 32, amx.GEMM_ROWS), got.contiguous())
    if K >= 512:
        assert amx.lib().amx_gemm_kernel_for(M, N, K, 32, amx.GEMM_AUTO) == amx.GEMM_ROWS
    fused = amx.quant_gemm(dev_bf16(a_bits), dev[2], dev[3], 32, flags=amx.GEMM_ROWS)
    assert torch.equal(fused, got.contiguous())


@pytest.mark.parametrize("rows", [13, 29, 61])
def test_gemm_rows_exact_on_small_integers(rows):
    """Integer-valued operands: every product and partial sum is exact in fp32, so any summation order gives the
    integer result - an independent check of the fragment order and the K ranges."""
    rng = np.random.default_rng(11)
    grid = np.array([0, 1, 2, 3, 4, 6], np.float32)
    def ints(r, k):
        t = grid[rng.integers(0, 6, size=(r, k))] * rng.choice([-1.0, 1.0], size=(r, k)).astype(np.float32)
        t[:, ::32], t[:, 1::32] = 6.0, -6.0
        return t
    a, w = ints(rows, 2304), ints(300, 2304)
    qa, qw = oracle.quantize(inputs.f32_to_bf16_bits(a), 32), oracle.quantize(inputs.f32_to_bf16_bits(w), 32)
    got = amx.gemm(*(torch.from_numpy(t).cuda() for t in (*qa, *qw)), 32, amx.GEMM_ROWS).cpu().numpy()
    assert np.array_equal(got, (a.astype(np.int64) @ w.astype(np.int64).T).astype(np.float32))


@pytest.mark.parametrize("fmt", [amx.FMT_AMXFP4, amx.FMT_SYM_FP8, amx.FMT_MXFP4])
@pytest.mark.parametrize("gs", [16, 32, 64, 128])
def test_quant_error_against_oracle(fmt, gs):
    """Error split (max-clamping / rounding) of every format and group size: the clamped count is exact, the sums
    agree with the oracle's fp64 sums to 2^-20 relative (the kernel adds the 16 non-negative squares of a chunk in
    fp32: at most 16 roundings of 2^-24 each), and two runs give the same bits.  Ragged shape (rows and K
    not multiples of the block's work), strided rows, inputs with clamping (power-of-two floor) and wide range."""
    for kind, rows, K in (("normal", 37, 1152), ("mixed", 5, 256), ("normal", 300, 4096)):
        bits = inputs.random_groups(1200 + gs + rows, rows, K, kind)
        wide = torch.zeros((rows, K + 64), dtype=torch.bfloat16, device="cuda")
        wide[:, :K] = dev_bf16(bits)
        x = wide[:, :K]
        codes, scales = amx.quantize(x, gs, fmt)
        ref = oracle.quant_error(bits, codes.cpu().numpy(), scales.cpu().numpy(), gs)
        got = amx.quant_error(x, codes, scales, gs)
        g = got.cpu().numpy()
        assert g[3] == ref[3]
        assert np.allclose(g[:3], ref[:3], rtol=2.0 ** -20, atol=0)
        assert torch.equal(amx.quant_error(x, codes, scales, gs), got)
    empty = amx.quant_error(x[:0], codes[:0], scales[:0], gs)
    assert torch.all(empty == 0)


def test_fp4_path_shape_sweep():
    """Seeded sweep of ragged shapes through the fused cast and the FP4 kernel (prepared buffers pre-filled with
    0xFF, padded output), against the oracle on the oracle's own codes."""
    rng = np.random.default_rng(2411)
    for case in range(10):
        M, N = int(rng.integers(1, 400)), int(rng.integers(1, 600))
        K = 32 * int(rng.integers(1, 72))
        fmt, mode = [(amx.FMT_AMXFP4, 0), (amx.FMT_SYM_FP8, oracle.SYMMETRIC_FP8), (amx.FMT_MXFP4, oracle.MXFP4)][case % 3]
        a_bits = inputs.random_groups(500 + case, M, K, "mixed" if case % 2 else "normal")
        w_bits = inputs.random_groups(600 + case, N, K, "normal")
        quant = (lambda b: oracle.quantize(b, 32)) if mode == 0 else (lambda b: oracle.quantize_variant(b, 32, mode))
        qa, qw = quant(a_bits), quant(w_bits)
        dirty = lambda rows, w: torch.full((amx.lib().amx_prepared_bytes(rows, K, 32, w),), 0xFF, dtype=torch.uint8, device="cuda")
        ac, as_, pa = amx.quantize_prepared(dev_bf16(a_bits), False, prepared=dirty(M, 0), fmt=fmt)
        wc, ws, pw = amx.quantize_prepared(dev_bf16(w_bits), True, prepared=dirty(N, 1), fmt=fmt)
        assert np.array_equal(ac.cpu().numpy(), qa[0]) and np.array_equal(as_.cpu().numpy(), qa[1]), (case, M, K)
        assert np.array_equal(wc.cpu().numpy(), qw[0]) and np.array_equal(ws.cpu().numpy(), qw[1]), (case, N, K)
        wide = torch.full((M, N + 5), -3.0, dtype=torch.float32, device="cuda")
        got = amx.gemm_prepared(pa, pw, M, N, K, out=wide[:, :N])
        ref = oracle.gemm(*qa, *qw, 32)
        if np.linalg.norm(ref) > 0:
            assert rel_fro(got.cpu().numpy(), ref) <= 2e-4, (case, M, N, K, fmt)
        assert torch.all(wide[:, N:] == -3.0)


def test_quantize_prepared_equals_quantize_then_prepare():
    # row lengths below, at and above one block of the cast kernel (several rows, one row and a fraction of a
    # row per block; threads striding over a long row), ragged row counts, both paddings
    cases = ((300, 1056, False, "mixed"), (520, 1056, True, "wide"), (130, 96, True, "mixed"), (8, 32, False, "normal"),
             (77, 11008, False, "mixed"), (20, 16448, True, "mixed"), (129, 4096, True, "wide"))
    for rows, K, is_w, kind in cases:
        bits = inputs.random_groups(63, rows, K, kind)
        x = dev_bf16(bits)
        # a buffer full of 0xFF: every byte the GEMM reads must have been written by the call
        dirty = torch.full((amx.lib().amx_prepared_bytes(rows, K, 32, int(is_w)),), 0xFF, dtype=torch.uint8, device="cuda")
        c, s_, prep = amx.quantize_prepared(x, is_w, prepared=dirty)
        c2, s2 = amx.quantize(x, 32)
        assert torch.equal(c, c2) and torch.equal(s_, s2)
        oc, os_ = oracle.quantize(bits, 32)
        assert np.array_equal(c.cpu().numpy(), oc) and np.array_equal(s_.cpu().numpy(), os_)
        # the prepared operands drive the GEMM to the same result
        w_bits = inputs.random_groups(64, 200, K, "normal")
        wc, ws = amx.quantize(dev_bf16(w_bits), 32)
        if is_w:
            other = amx.prepare(wc, ws, False)
            got = amx.gemm_prepared(other, prep, 200, rows, K)
            want = amx.gemm_prepared(other, amx.prepare(c2, s2, True), 200, rows, K)
        else:
            other = amx.prepare(wc, ws, True)
            got = amx.gemm_prepared(prep, other, rows, 200, K)
            want = amx.gemm_prepared(amx.prepare(c2, s2, False), other, rows, 200, K)
        assert torch.equal(got, want)


def test_gemm_wide_dynamic_range_rows():
    got, ref = _gemm_case(42, 96, 64, 256, 32, amx.GEMM_SIMT, "mixed")
    for m in range(96):                        # row-wise: rows differ by many orders of magnitude
        if np.all(np.isfinite(ref[m])) and np.linalg.norm(ref[m]) > 0:
            assert rel_fro(got[m], ref[m]) <= GEMM_TOL


def test_gemm_exact_on_small_integers():
    rng = np.random.default_rng(7)
    grid = np.array([0, 1, 2, 3, 4, 6], np.float32)
    def ints(r, k):
        t = grid[rng.integers(0, 6, size=(r, k))] * rng.choice([-1.0, 1.0], size=(r, k)).astype(np.float32)
        t[:, ::32], t[:, 1::32] = 6.0, -6.0
        return t
    a, w = ints(130, 256), ints(70, 256)
    qa, qw = oracle.quantize(inputs.f32_to_bf16_bits(a), 32), oracle.quantize(inputs.f32_to_bf16_bits(w), 32)
    got = amx.gemm(*(torch.from_numpy(t).cuda() for t in (*qa, *qw)), 32, amx.GEMM_SIMT).cpu().numpy()
    assert np.array_equal(got, (a.astype(np.int64) @ w.astype(np.int64).T).astype(np.float32))


def test_quant_gemm_equals_quantize_then_gemm():
    a = dev_bf16(inputs.activation(1, 0))
    wc, ws = amx.quantize(dev_bf16(inputs.weight(1, 0)), 32)
    ac, as_ = amx.quantize(a, 32)
    assert torch.equal(amx.quant_gemm(a, wc, ws, 32), amx.gemm(ac, as_, wc, ws, 32))


@pytest.mark.parametrize("M,N,K,kind", [(128, 512, 1024, "mixed"), (130, 300, 96, "wide"), (1, 8, 32, "normal"),
                                        (257, 260, 4096, "mixed")])
def test_quant_gemm_cast_in_kernel(M, N, K, kind):
    """The tensor-core kernel whose producers cast the activation tile themselves: bit-identical to
    amx_quantize followed by amx_gemm on the same kernel, and within tolerance of the oracle."""
    a_bits = inputs.random_groups(301 + M, M, K, kind)
    w_bits = inputs.random_groups(302 + N, N, K, "normal")
    a = dev_bf16(a_bits)
    wc, ws = amx.quantize(dev_bf16(w_bits), 32)
    ac, as_ = amx.quantize(a, 32)
    fused = amx.GEMM_TC | amx.GEMM_CAST_IN_KERNEL
    got = amx.quant_gemm(a, wc, ws, 32, flags=fused)
    assert torch.equal(got, amx.gemm(ac, as_, wc, ws, 32, flags=amx.GEMM_TC))
    ref = oracle.gemm(*oracle.quantize(a_bits, 32), wc.cpu().numpy(), ws.cpu().numpy(), 32)
    assert rel_fro(got.cpu().numpy(), ref) <= GEMM_TOL
    # a row-strided activation (a view into a wider buffer) gives the same result
    wide = torch.zeros((M, K + 64), dtype=torch.bfloat16, device="cuda")
    wide[:, 8:8 + K] = a
    assert torch.equal(amx.quant_gemm(wide[:, 8:8 + K], wc, ws, 32, flags=fused), got)


def test_config1_full_layer():
    a_bits, w_bits = inputs.activation(1, 0), inputs.weight(1, 0)
    ac, as_ = check_quantize(a_bits)
    wc, ws = check_quantize(w_bits)
    got = amx.gemm(ac, as_, wc, ws, 32).cpu().numpy()
    ref = oracle.gemm(ac.cpu().numpy(), as_.cpu().numpy(), wc.cpu().numpy(), ws.cpu().numpy(), 32)
    assert rel_fro(got, ref) <= GEMM_TOL


def test_linear_host_entry_point():
    a_bits, w_bits = inputs.activation(1, 0), inputs.weight(1, 0, N=256)
    a = torch.from_numpy(a_bits.view(np.int16)).view(torch.bfloat16).pin_memory()
    w = torch.from_numpy(w_bits.view(np.int16)).view(torch.bfloat16).pin_memory()
    c = torch.empty((128, 256), dtype=torch.float32).pin_memory()
    ws = torch.empty(amx.lib().amx_linear_host_workspace_bytes(128, 256, 1024, 32, 0), dtype=torch.uint8, device="cuda")
    amx.linear_host(a, w, c, ws)
    ref = oracle.gemm(*oracle.quantize(a_bits, 32), *oracle.quantize(w_bits, 32), 32)
    assert rel_fro(c.numpy(), ref) <= GEMM_TOL


# ----------------------------------------------------------- attention glue --

def test_softmax_bf16_against_oracle():
    rng = np.random.default_rng(8)
    S = (rng.standard_normal((40, 1000)) * 30).astype(np.float32)
    got = amx.softmax_bf16(torch.from_numpy(S).cuda(), 128 ** -0.5).view(torch.int16).cpu().numpy().view(np.uint16)
    want = oracle.softmax_bf16(S, 128 ** -0.5)
    # fp32 exp on the device vs fp64 exp on the host: allow one bf16 ulp on a small fraction
    diff = np.abs(got.astype(np.int32) - want.astype(np.int32))
    assert diff.max() <= 1 and np.mean(diff != 0) < 0.02


@pytest.mark.parametrize("rows,cols,scale", [(40, 1024, 30.0), (130, 96, 3.0), (9, 8192, 50.0), (5, 8224, 8.0),
                                             (3, 32, 1.0)])
def test_softmax_quantize_fused_equals_two_kernels(rows, cols, scale):
    """amx_softmax_quantize: same bits as amx_softmax_bf16 followed by amx_quantize; the oracle quantizer on the
    device's own bf16 map gives the same codes and scales; the prepared form drives the GEMM to the same result.
    Rows of at most 8192 columns take the register-cached path, longer ones the re-reading one."""
    rng = np.random.default_rng(80 + rows)
    S_np = (rng.standard_normal((rows, cols)) * scale).astype(np.float32)
    S_np[0, : cols // 2] = -1e4                              # half a row underflows to exactly zero
    S = torch.from_numpy(S_np).cuda()
    alpha = 128 ** -0.5
    P = amx.softmax_bf16(S, alpha)
    c2, s2 = amx.quantize(P, 32)
    c, s_ = amx.softmax_quantize(S, alpha)
    assert torch.equal(c, c2) and torch.equal(s_, s2)
    oc, os_ = oracle.quantize(P.view(torch.int16).cpu().numpy().view(np.uint16), 32)
    assert np.array_equal(c.cpu().numpy(), oc) and np.array_equal(s_.cpu().numpy(), os_)
    # strided logits (a view into a wider buffer)
    wide = torch.zeros((rows, cols + 40), dtype=torch.float32, device="cuda")
    wide[:, 4:4 + cols] = S
    cw, sw = amx.softmax_quantize(wide[:, 4:4 + cols], alpha)
    assert torch.equal(cw, c) and torch.equal(sw, s_)
    wide[:, 1:1 + cols] = S                                   # rows not 16-byte aligned: scalar loads
    cw, sw = amx.softmax_quantize(wide[:, 1:1 + cols], alpha)
    assert torch.equal(cw, c) and torch.equal(sw, s_)
    # prepared form, as the left-hand operand of P V
    cp, sp, prep = amx.softmax_quantize(S, alpha, prepared_as="a")
    assert torch.equal(cp, c) and torch.equal(sp, s_)
    v_bits = inputs.random_groups(81, 64, cols, "normal")
    vc, vs = amx.quantize(dev_bf16(v_bits), 32)
    pv = amx.prepare(vc, vs, True)
    assert torch.equal(amx.gemm_prepared(prep, pv, rows, 64, cols),
                       amx.gemm_prepared(amx.prepare(c2, s2, False), pv, rows, 64, cols))


def test_attention_small_head_against_oracle_pipeline():
    """Config-5 pipeline at reduced size: Q/K/V codes bit-exact; the device quantizer applied to the
    device's own bf16 P equals the oracle quantizer on the same bits; O within tolerance of the all-CPU
    pipeline."""
    qb, kb, vb = (t[0] for t in inputs.attention_qkv(heads=1, seq=256))
    O, P = amx.attention(dev_bf16(qb), dev_bf16(kb), dev_bf16(vb))
    check_quantize(qb), check_quantize(kb)
    vc, vs = amx.quantize_t(dev_bf16(vb), 32)
    ovc, ovs = oracle.quantize(np.ascontiguousarray(vb.T), 32)
    assert np.array_equal(vc.cpu().numpy(), ovc) and np.array_equal(vs.cpu().numpy(), ovs)
    p_bits = P.view(torch.int16).cpu().numpy().view(np.uint16)
    check_quantize(p_bits)
    # all-CPU pipeline
    S = oracle.gemm(*oracle.quantize(qb, 32), *oracle.quantize(kb, 32), 32)
    Pcpu = oracle.softmax_bf16(S, 128 ** -0.5)
    Ocpu = oracle.gemm(*oracle.quantize(Pcpu, 32), ovc, ovs, 32)
    assert rel_fro(O.cpu().numpy(), Ocpu) <= GEMM_TOL


@pytest.mark.parametrize("heads,seq,flags", [(3, 320, amx.GEMM_AUTO),      # head by head (seq % 128 != 0)
                                             (10, 128, amx.GEMM_AUTO),     # chunks of 8 + 2 heads, small-product kernel
                                             (9, 256, amx.GEMM_FP4),       # chunks of 8 + 1, FP4 kernel on stacked operands
                                             (2, 1024, amx.GEMM_AUTO)])    # AUTO picks the FP4 kernel
def test_attention_all_heads_entry_point_matches_per_head_pipeline(heads, seq, flags):
    q, k, v = (dev_bf16(t) for t in inputs.attention_qkv(heads=heads, seq=seq))
    O = amx.attention_heads(q, k, v, flags=flags)
    fused = seq % 128 == 0 and amx.lib().amx_gemm_kernel_for(seq, seq, 128, 32, flags) == amx.GEMM_FP4
    for h in range(heads):
        Oh, _ = amx.attention(q[h], k[h], v[h], flags=flags)
        if fused:
            # fused kernel: the row sums are taken tile by tile, in another order than the one-kernel softmax of the
            # per-head pipeline, so a few elements of P round to the neighbouring bf16 value
            assert rel_fro(O[h].cpu().numpy(), Oh.cpu().numpy()) <= 1e-4, h
        else:
            assert torch.equal(O[h], Oh), h


@pytest.mark.parametrize("heads,seq,flags", [(2, 192, amx.GEMM_AUTO),        # stored logits, small-product kernel
                                             (1, 320, amx.GEMM_FP4),         # stored logits, FP4 kernel
                                             (2, 512, amx.GEMM_FP4),         # fused kernel, key blocks after the queries skipped
                                             (1, 1024, amx.GEMM_AUTO)])
def test_attention_causal_against_oracle_pipeline(heads, seq, flags):
    """Causal attention (query i sees keys 0..i) against the all-CPU pipeline with the mask applied before the
    softmax, every query row; the first query returns V's first row as quantized, times the quantized 1."""
    qb, kb, vb = inputs.attention_qkv(heads=heads, seq=seq)
    O = amx.attention_heads(dev_bf16(qb), dev_bf16(kb), dev_bf16(vb), flags=flags | amx.ATTN_CAUSAL).cpu().numpy()
    assert np.all(np.isfinite(O))
    for h in range(heads):
        S = oracle.gemm(*oracle.quantize(qb[h], 32), *oracle.quantize(kb[h], 32), 32)
        P = oracle.softmax_bf16(S, 128 ** -0.5, causal_row0=0)
        vq = oracle.quantize(np.ascontiguousarray(vb[h].T), 32)
        ref = oracle.gemm(*oracle.quantize(P, 32), *vq, 32)
        assert rel_fro(O[h], ref) <= GEMM_TOL, h
        # the first query sees one key: P = 1 there, which AMXFP4 stores as 6 x 0.15625 (scale nearest to 1/6)
        assert np.allclose(O[h][0], 0.9375 * oracle.dequantize(*vq, 32)[:, 0], rtol=1e-6, atol=0)


def test_attention_fused_kernel_against_oracle_pipeline():
    """Attention in the fused kernel (FP4 kernel forced, head dimension 128, sequence a multiple of 128): output
    against the all-CPU pipeline, every query row."""
    qb, kb, vb = (t[0] for t in inputs.attention_qkv(heads=1, seq=512))
    O = amx.attention_heads(dev_bf16(qb)[None], dev_bf16(kb)[None], dev_bf16(vb)[None], flags=amx.GEMM_FP4)[0]
    S = oracle.gemm(*oracle.quantize(qb, 32), *oracle.quantize(kb, 32), 32)
    P = oracle.softmax_bf16(S, 128 ** -0.5)
    ref = oracle.gemm(*oracle.quantize(P, 32), *oracle.quantize(np.ascontiguousarray(vb.T), 32), 32)
    assert rel_fro(O.cpu().numpy(), ref) <= GEMM_TOL


def test_config5_full_size_attention_sampled():
    """32 heads x 8192 tokens x 128: every head through amx_attention; heads 0 and 31 checked against the
    all-CPU pipeline on sampled query rows, and the device quantizer against the oracle on the device's own
    bf16 attention map."""
    qb, kb, vb = inputs.attention_qkv()
    q, k, v = dev_bf16(qb), dev_bf16(kb), dev_bf16(vb)
    O = amx.attention_heads(q, k, v).cpu().numpy()
    assert np.all(np.isfinite(O))
    rng = np.random.default_rng(55)
    for h in (0, 31):
        rows = np.sort(rng.choice(8192, size=48, replace=False))
        qc, qs = oracle.quantize(qb[h][rows], 32)
        kc, ks = oracle.quantize(kb[h], 32)
        vc, vs = oracle.quantize(np.ascontiguousarray(vb[h].T), 32)
        S = oracle.gemm(qc, qs, kc, ks, 32)
        P = oracle.softmax_bf16(S, 128 ** -0.5)
        ref = oracle.gemm(*oracle.quantize(P, 32), vc, vs, 32)
        assert rel_fro(O[h][rows], ref) <= GEMM_TOL, h
    # the device quantizer on the device's own attention map (head 0), sampled rows
    _, Pdev = amx.attention(q[0], k[0], v[0])
    pc, ps = amx.quantize(Pdev, 32)
    rows = np.sort(rng.choice(8192, size=256, replace=False))
    p_bits = Pdev[torch.from_numpy(rows).cuda()].view(torch.int16).cpu().numpy().view(np.uint16)
    opc, ops = oracle.quantize(p_bits, 32)
    assert np.array_equal(pc.cpu().numpy()[rows], opc) and np.array_equal(ps.cpu().numpy()[rows], ops)


@pytest.mark.parametrize("causal", [False, True])
def test_attention_long_sequence_sampled(causal):
    """Twice config 5's sequence length (16384 tokens, the fused kernel, logits and map never stored): sampled query
    rows against the all-CPU pipeline."""
    L = 16384
    qb, kb, vb = (t[0] for t in inputs.attention_qkv(heads=1, seq=L))
    O = amx.attention_heads(dev_bf16(qb)[None], dev_bf16(kb)[None], dev_bf16(vb)[None],
                            flags=amx.ATTN_CAUSAL if causal else 0)[0].cpu().numpy()
    assert np.all(np.isfinite(O))
    rows = np.sort(np.random.default_rng(56).choice(L, size=32, replace=False))
    S = oracle.gemm(*oracle.quantize(qb[rows], 32), *oracle.quantize(kb, 32), 32)
    if causal:
        for i, r in enumerate(rows):
            S[i, r + 1:] = -np.inf
    P = oracle.softmax_bf16(S, 128 ** -0.5)
    ref = oracle.gemm(*oracle.quantize(P, 32), *oracle.quantize(np.ascontiguousarray(vb.T), 32), 32)
    assert rel_fro(O[rows], ref) <= GEMM_TOL


# ------------------------------------------------ full-size configurations --

@pytest.mark.parametrize("config,layer", [(c, l) for c in (2, 3, 4) for l in range(len(inputs.LINEAR_CONFIGS[c]["layers"]))])
def test_full_size_layer_sampled(config, layer):
    """Every layer of the three large configurations at its full size, whole-tensor launches.  Codes and scales are
    compared on the whole activation for config 2 and on sampled rows otherwise; the product on 64 sampled rows x
    all N, for amx_gemm and for the launch sequence the benchmark times (casts that write the FP4 kernel's
    operands, then the GEMM on them), whose status word and flushed-scale counts are checked too."""
    spec = inputs.LINEAR_CONFIGS[config]
    M = spec["M"]
    a_bits, w_bits = inputs.activation(config, layer), inputs.weight(config, layer)
    K, N = a_bits.shape[1], w_bits.shape[0]
    a, w = dev_bf16(a_bits), dev_bf16(w_bits)
    ac, as_ = amx.quantize(a, 32)
    wc, ws = amx.quantize(w, 32)
    rng = np.random.default_rng(100 * config + layer)
    rows = np.sort(rng.choice(M, size=64, replace=False))
    rows_dev = torch.from_numpy(rows).cuda()
    arow = np.arange(M) if config == 2 else np.union1d(rows, rng.choice(M, size=256, replace=False))
    arow_dev = torch.from_numpy(arow).cuda()
    oac, oas = oracle.quantize(a_bits[arow], 32)
    assert np.array_equal(ac[arow_dev].cpu().numpy(), oac) and np.array_equal(as_[arow_dev].cpu().numpy(), oas)
    wrow = np.sort(rng.choice(N, size=512, replace=False))
    wrow_dev = torch.from_numpy(wrow).cuda()
    owc, ows = oracle.quantize(w_bits[wrow], 32)
    assert np.array_equal(wc[wrow_dev].cpu().numpy(), owc) and np.array_equal(ws[wrow_dev].cpu().numpy(), ows)
    # reference on the sampled rows: the oracle's own codes of those rows against the device's weight codes
    # (checked above on a sample; the product below would expose a wrong row anywhere else)
    sel = np.searchsorted(arow, rows)
    ref = oracle.gemm(oac[sel], oas[sel], wc.cpu().numpy(), ws.cpu().numpy(), 32)
    got = amx.gemm(ac, as_, wc, ws, 32)[rows_dev].cpu().numpy()
    assert rel_fro(got, ref) <= GEMM_TOL
    del got
    # the launch sequence the benchmark times
    ac2, as2, pa = amx.quantize_prepared(a, False)
    wc2, ws2, pw = amx.quantize_prepared(w, True)
    assert torch.equal(ac2, ac) and torch.equal(as2, as_) and torch.equal(wc2, wc) and torch.equal(ws2, ws)
    assert amx.prepared_flushed_scales(pa, M, K, False) == 0 and amx.prepared_flushed_scales(pw, N, K, True) == 0
    work = torch.empty(256, dtype=torch.uint8, device="cuda")
    got2 = amx.gemm_prepared(pa, pw, M, N, K, workspace=work)[rows_dev].cpu().numpy()
    assert amx.gemm_status(work) == 0
    assert rel_fro(got2, ref) <= GEMM_TOL
