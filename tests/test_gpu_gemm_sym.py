"""GPU parity of the one-plane form of the FP4 tensor-core GEMM (amx_gemm_prepared_sym, amx_gemm_nvfp4_sym) and of the
options of amx_gemm_prepared_ex (one plane, bf16 result); products with several tiles per persistent CTA.  Two
operands in a symmetric comparison format (Section 5's MXFP4 and FP8-scaled baselines, NVFP4) need one product per K
step.  The result must equal the general kernel's bit for bit (same MMAs in the same order on the same scale factors)
and the CPU oracle's within the GEMM tolerance; an operand with two planes must show as AMX_ERR_FLAGS in the status."""
import numpy as np
import pytest
import torch

import oracle
from paper_2411_09909_b200 import amx, inputs

pytestmark = pytest.mark.gpu

GEMM_TOL = 1e-3          # relative Frobenius error against the oracle's fp64 product (fp32 accumulation)
ERR_FLAGS = -5


def dev_bf16(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def rel_fro(got, ref):
    return np.linalg.norm(got.astype(np.float64) - ref) / max(np.linalg.norm(ref), 1e-300)


def fresh_ws(M, N, K):
    return torch.full((amx.lib().amx_gemm_prepared_workspace_bytes(M, N, K, 32),), 0xFF, dtype=torch.uint8, device="cuda")


FORMATS = [(amx.FMT_SYM_FP8, oracle.SYMMETRIC_FP8), (amx.FMT_MXFP4, oracle.MXFP4)]


@pytest.mark.parametrize("fmt,mode", FORMATS)
@pytest.mark.parametrize("M,N,K", [(300, 520, 1056), (400, 777, 2080), (129, 257, 32), (1, 300, 64), (128, 256, 4096)])
def test_gemm_prepared_sym_against_oracle_and_general_kernel(fmt, mode, M, N, K):
    a_bits = inputs.random_groups(4100 + M, M, K, "mixed" if M % 2 else "normal")
    w_bits = inputs.random_groups(4200 + N, N, K, "normal")
    qa, qw = oracle.quantize_variant(a_bits, 32, mode), oracle.quantize_variant(w_bits, 32, mode)
    ac, as_, pa = amx.quantize_prepared(dev_bf16(a_bits), False, fmt=fmt)
    wc, ws_, pw = amx.quantize_prepared(dev_bf16(w_bits), True, fmt=fmt)
    assert np.array_equal(ac.cpu().numpy(), qa[0]) and np.array_equal(as_.cpu().numpy(), qa[1])
    assert np.array_equal(wc.cpu().numpy(), qw[0]) and np.array_equal(ws_.cpu().numpy(), qw[1])
    work = fresh_ws(M, N, K)
    wide = torch.full((M, N + 3), -3.0, dtype=torch.float32, device="cuda")
    got = amx.gemm_prepared(pa, pw, M, N, K, out=wide[:, :N], workspace=work, sym=True)
    assert amx.gemm_status(work) == 0
    assert torch.all(wide[:, N:] == -3.0)
    general = amx.gemm_prepared(pa, pw, M, N, K)
    assert torch.equal(got, general)
    ref = oracle.gemm(*qa, *qw, 32)
    if np.linalg.norm(ref) > 0:
        assert rel_fro(got.cpu().numpy(), ref) <= GEMM_TOL


def test_gemm_prepared_sym_full_size_layer():
    """Config 2's first layer (2048 x 4096 -> 12288) in MXFP4: equal to the general kernel everywhere (several waves of
    tiles per CTA, 32 K blocks through the 8 stages), 48 sampled rows against the oracle."""
    a_bits, w_bits = inputs.activation(2, 0), inputs.weight(2, 0)
    M, K, N = 2048, 4096, 12288
    _, _, pa = amx.quantize_prepared(dev_bf16(a_bits), False, fmt=amx.FMT_MXFP4)
    wc, ws_, pw = amx.quantize_prepared(dev_bf16(w_bits), True, fmt=amx.FMT_MXFP4)
    work = fresh_ws(M, N, K)
    got = amx.gemm_prepared(pa, pw, M, N, K, workspace=work, sym=True)
    assert amx.gemm_status(work) == 0
    assert torch.equal(got, amx.gemm_prepared(pa, pw, M, N, K))
    rows = np.sort(np.random.default_rng(41).choice(M, size=48, replace=False))
    qa = oracle.quantize_variant(a_bits[rows], 32, oracle.MXFP4)
    ref = oracle.gemm(*qa, wc.cpu().numpy(), ws_.cpu().numpy(), 32)
    assert rel_fro(got[torch.from_numpy(rows).cuda()].cpu().numpy(), ref) <= GEMM_TOL


@pytest.mark.parametrize("fmt,mode", [(amx.FMT_AMXFP4, 0), (amx.FMT_MXFP4, oracle.MXFP4)])
@pytest.mark.parametrize("M,N,K", [(1100, 6200, 1056), (2304, 6400, 288), (130, 40000, 160)])
def test_several_tiles_per_cta(fmt, mode, M, N, K):
    """Products whose persistent CTAs get one and two, three and four, and two tiles each (225, 450 and 314 tiles on
    148 CTAs): consecutive tiles of a CTA alternate between the two accumulator windows.  Two rows of every block of
    128 rows against the oracle, so that every output tile is checked; the general and the one-plane kernel."""
    a_bits = inputs.random_groups(4700 + M, M, K, "normal")
    w_bits = inputs.random_groups(4800 + M, N, K, "normal")
    quant = (lambda b: oracle.quantize(b, 32)) if mode == 0 else (lambda b: oracle.quantize_variant(b, 32, mode))
    _, _, pa = amx.quantize_prepared(dev_bf16(a_bits), False, fmt=fmt)
    wc, ws_, pw = amx.quantize_prepared(dev_bf16(w_bits), True, fmt=fmt)
    rng = np.random.default_rng(47)
    rows = np.sort(np.concatenate([b + rng.choice(min(128, M - b), size=2, replace=False) for b in range(0, M, 128)]))
    qa = quant(a_bits[rows])
    ref = oracle.gemm(*qa, wc.cpu().numpy(), ws_.cpu().numpy(), 32)
    rows_dev = torch.from_numpy(rows).cuda()
    for sym in ([False, True] if mode else [False]):
        work = torch.full((256,), 0xFF, dtype=torch.uint8, device="cuda")
        got = amx.gemm_prepared(pa, pw, M, N, K, workspace=work, sym=sym)
        assert amx.gemm_status(work) == 0
        assert rel_fro(got[rows_dev].cpu().numpy(), ref) <= GEMM_TOL
        # no tile differs from the rest: per-tile error norms against the exact bf16-decode kernel's product
        if not sym and mode == 0:
            ac, as_ = amx.quantize(dev_bf16(a_bits), 32)
            exact = amx.gemm(ac, as_, wc, ws_, 32, amx.GEMM_TC)
            err = (got - exact).abs().amax(dim=0).cpu().numpy(), exact.abs().amax().item()
            assert err[0].max() <= 1e-4 * err[1]


def test_one_signed_amxfp4_operand_is_a_single_plane():
    """An AMXFP4 operand whose values are all non-negative (an activation after ReLU) has no negative plane."""
    M, N, K = 260, 515, 1024
    a_bits = inputs.random_groups(4301, M, K, "normal") & np.uint16(0x7FFF)
    w_bits = inputs.random_groups(4302, N, K, "normal")
    qa, qw = oracle.quantize(a_bits, 32), oracle.quantize_variant(w_bits, 32, oracle.SYMMETRIC_FP8)
    _, _, pa = amx.quantize_prepared(dev_bf16(a_bits), False)
    _, _, pw = amx.quantize_prepared(dev_bf16(w_bits), True, fmt=amx.FMT_SYM_FP8)
    work = fresh_ws(M, N, K)
    got = amx.gemm_prepared(pa, pw, M, N, K, workspace=work, sym=True)
    assert amx.gemm_status(work) == 0
    assert rel_fro(got.cpu().numpy(), oracle.gemm(*qa, *qw, 32)) <= GEMM_TOL


@pytest.mark.parametrize("which", ["a", "w", "one row"])
def test_two_plane_operand_is_reported(which):
    M, N, K = 300, 520, 1056
    a_bits = inputs.random_groups(4401, M, K, "normal")
    w_bits = inputs.random_groups(4402, N, K, "normal")
    fa = amx.FMT_AMXFP4 if which == "a" else amx.FMT_SYM_FP8
    fw = amx.FMT_AMXFP4 if which == "w" else amx.FMT_SYM_FP8
    if which == "one row":                  # a single row of W in the last tile with differing scales
        wq = list(oracle.quantize_variant(w_bits, 32, oracle.SYMMETRIC_FP8))
        wq[0], wq[1] = wq[0].copy(), wq[1].copy()
        amx_row = oracle.quantize(w_bits[N - 1:N], 32)
        wq[0][N - 1], wq[1][N - 1] = amx_row[0][0], amx_row[1][0]
        assert not np.array_equal(wq[1][N - 1, :, 0], wq[1][N - 1, :, 1])
        pw = amx.prepare(torch.from_numpy(wq[0]).cuda(), torch.from_numpy(wq[1]).cuda(), True)
    else:
        _, _, pw = amx.quantize_prepared(dev_bf16(w_bits), True, fmt=fw)
    _, _, pa = amx.quantize_prepared(dev_bf16(a_bits), False, fmt=fa)
    work = fresh_ws(M, N, K)
    amx.gemm_prepared(pa, pw, M, N, K, workspace=work, sym=True)
    assert amx.gemm_status(work) == ERR_FLAGS
    # the general kernel on the same operands and workspace afterwards is unaffected
    got = amx.gemm_prepared(pa, pw, M, N, K, workspace=work)
    assert amx.gemm_status(work) == 0
    assert torch.isfinite(got).all()


@pytest.mark.parametrize("M,N,K", [(300, 520, 1088), (128, 256, 64), (1, 1, 64), (515, 1030, 2048)])
def test_gemm_nvfp4_sym(M, N, K):
    a_bits = inputs.random_groups(4500 + M, M, K, "normal")
    w_bits = inputs.random_groups(4501 + N, N, K, "normal")
    qa, qw = oracle.quantize_nv(a_bits, False), oracle.quantize_nv(w_bits, False)
    _, _, _, pa = amx.quantize_nvfp4(dev_bf16(a_bits), False, prepared_as="a")
    _, _, _, pw = amx.quantize_nvfp4(dev_bf16(w_bits), False, prepared_as="w")
    work = torch.full((256,), 0xFF, dtype=torch.uint8, device="cuda")
    got = amx.gemm_nvfp4(pa, pw, M, N, K, workspace=work, sym=True)
    assert amx.gemm_status(work) == 0
    assert torch.equal(got, amx.gemm_nvfp4(pa, pw, M, N, K))
    assert rel_fro(got.cpu().numpy(), oracle.gemm_nv(*qa, *qw)) <= 1e-5
    # ANVFP4 against the promise
    _, _, _, pa2 = amx.quantize_nvfp4(dev_bf16(a_bits), True, prepared_as="a")
    amx.gemm_nvfp4(pa2, pw, M, N, K, workspace=work, sym=True)
    two_planes = bool(np.any(a_bits & 0x8000) and np.any((a_bits & 0x8000) == 0) and N > 128)
    assert amx.gemm_status(work) == (ERR_FLAGS if two_planes else 0)


@pytest.mark.parametrize("sym", [False, True])
@pytest.mark.parametrize("M,N,K,pad", [(300, 520, 1056, 8), (129, 257, 64, 3), (1100, 6200, 288, 0), (1, 16, 32, 0), (128, 256, 4096, 0)])
def test_bf16_result(sym, M, N, K, pad):
    """amx_gemm_prepared_ex with AMX_PREP_OUT_BF16: the fp32 result of the same kernel rounded to bf16 (ties to even), bit
    for bit; vector and scalar store paths (leading dimension a multiple of 16 or not), padding untouched."""
    fmt = amx.FMT_MXFP4 if sym else amx.FMT_AMXFP4
    a_bits = inputs.random_groups(4900 + M, M, K, "normal")
    w_bits = inputs.random_groups(4950 + N, N, K, "normal")
    _, _, pa = amx.quantize_prepared(dev_bf16(a_bits), False, fmt=fmt)
    _, _, pw = amx.quantize_prepared(dev_bf16(w_bits), True, fmt=fmt)
    work = torch.full((256,), 0xFF, dtype=torch.uint8, device="cuda")
    f32 = amx.gemm_prepared(pa, pw, M, N, K, workspace=work, sym=sym)
    wide = torch.full((M, N + pad), -3.0, dtype=torch.bfloat16, device="cuda")
    got = amx.gemm_prepared(pa, pw, M, N, K, out=wide[:, :N], workspace=work, sym=sym)
    assert amx.gemm_status(work) == 0
    assert got.dtype == torch.bfloat16 and torch.equal(got, f32.to(torch.bfloat16))      # torch rounds to nearest even
    assert torch.all(wide[:, N:] == -3.0)
    L = amx.lib()
    st = torch.cuda.current_stream().cuda_stream
    assert L.amx_gemm_prepared_ex(pa.data_ptr(), pw.data_ptr(), M, N, K, 32, 0x4, wide.data_ptr(), N + pad, work.data_ptr(), 256, st) == -5
    assert L.amx_gemm_prepared_ex(pa.data_ptr(), pw.data_ptr(), M, N, K, 32, 0x2, wide.data_ptr() + 1, N + pad, work.data_ptr(), 256, st) == -3
    # a workspace that would allow K ranges changes nothing: a bf16 result is never assembled from partial sums
    big = torch.empty(L.amx_gemm_prepared_workspace_bytes(M, N, K, 32), dtype=torch.uint8, device="cuda")
    assert torch.equal(amx.gemm_prepared(pa, pw, M, N, K, workspace=big, sym=sym, out_dtype=torch.bfloat16), got)
    # without flags: amx_gemm_prepared
    c = torch.empty((M, N), dtype=torch.float32, device="cuda")
    assert L.amx_gemm_prepared_ex(pa.data_ptr(), pw.data_ptr(), M, N, K, 32, 0, c.data_ptr(), N, work.data_ptr(), 256, st) == 0
    assert torch.equal(c, amx.gemm_prepared(pa, pw, M, N, K, workspace=work))


def test_sym_argument_errors():
    L = amx.lib()
    buf = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    c = torch.zeros((128, 256), dtype=torch.float32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    p, w = buf.data_ptr(), buf.data_ptr() + (1 << 19)
    assert L.amx_gemm_prepared_sym(p, w, 128, 256, 64, 16, c.data_ptr(), 256, w, 256, st) == -2
    assert L.amx_gemm_prepared_sym(None, w, 128, 256, 64, 32, c.data_ptr(), 256, w, 256, st) == -1
    assert L.amx_gemm_prepared_sym(p, w, 128, 256, 64, 32, c.data_ptr(), 256, None, 0, st) == -4
    assert L.amx_gemm_prepared_sym(p + 16, w, 128, 256, 64, 32, c.data_ptr(), 256, w, 256, st) == -3
    assert L.amx_gemm_nvfp4_sym(p, w, 128, 256, 96, c.data_ptr(), 256, w, 256, st) == -2
    assert L.amx_gemm_nvfp4_sym(p, None, 128, 256, 64, c.data_ptr(), 256, w, 256, st) == -1
    torch.cuda.synchronize()
