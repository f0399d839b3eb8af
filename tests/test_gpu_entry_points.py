"""GPU tests of the boundary's less travelled entry points: the one-call layer with a bf16 weight (both operands
cast per call), whole-row groups through the generic kernels (the paper's worked example), the status word after
every kernel choice, the bounded-wait self-test, and the host-buffer layer with an explicit kernel."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2411_09909_b200 import amx, inputs

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_example.txt")


def dev_bf16(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def rel_fro(got, ref):
    return np.linalg.norm(got.astype(np.float64) - ref) / np.linalg.norm(ref)


def _golden():
    out = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        name, *vals = line.split()
        out[name] = [float(v) for v in vals]
    return out


def test_worked_example_through_the_library():
    """Appendix B.3: x = linspace(-4.9, 31, 1024) cast to bf16, the whole row one group.  The three value sets the
    paper prints come back from amx_quantize_fmt + amx_dequantize, and the codes and scales equal the oracle's."""
    x = torch.linspace(-4.9, 31, 1024, dtype=torch.float32).to(torch.bfloat16)
    bits = x.view(torch.int16).numpy().view(np.uint16)[None, :].copy()
    gold = _golden()
    for name, fmt, mode in (("amxfp4_fp8", amx.FMT_AMXFP4, None), ("mxfp4_pot", amx.FMT_MXFP4, oracle.MXFP4),
                            ("amxfp4_pot", amx.FMT_AMXFP4_POT, oracle.AMXFP4_POT)):
        c, s = amx.quantize(dev_bf16(bits), 1024, fmt=fmt)
        assert s.shape == (1, 1, 2)
        oc, os_ = oracle.quantize(bits, 1024) if mode is None else oracle.quantize_variant(bits, 1024, mode)
        assert np.array_equal(c.cpu().numpy(), oc) and np.array_equal(s.cpu().numpy(), os_), name
        vals = amx.dequantize(c, s, 1024, torch.float32).double().cpu().numpy()
        assert sorted(set(vals.ravel())) == gold[name], name
    c, s = amx.quantize(dev_bf16(bits), 1024)
    assert oracle.e5m2_value(int(s[0, 0, 0])) == 5.0 and oracle.e5m2_value(int(s[0, 0, 1])) == 0.875
    d = amx.dequantize(c, s, 1024, torch.float32).cpu().numpy()
    assert d[0, -1] == 30.0 and d[0, 0] == -5.25


@pytest.mark.parametrize("rows,K", [(37, 1000), (3, 8), (130, 4104)])
def test_whole_row_groups_quantize_dequantize_gemm(rows, K):
    """group_size == K on the generic kernels, ragged sizes and strided rows."""
    bits = inputs.random_groups(1700 + rows, rows, (K + 31) // 32 * 32, "mixed")[:, :K].copy()
    wide = torch.zeros((rows, K + 24), dtype=torch.bfloat16, device="cuda")
    wide[:, 8:8 + K] = dev_bf16(bits)
    c, s = amx.quantize(wide[:, 8:8 + K], K)
    oc, os_ = oracle.quantize(bits, K)
    assert np.array_equal(c.cpu().numpy(), oc) and np.array_equal(s.cpu().numpy(), os_)
    assert np.array_equal(amx.dequantize(c, s, K, torch.float32).double().cpu().numpy(), oracle.dequantize(oc, os_, K))
    w_bits = inputs.random_groups(1800 + rows, 70, (K + 31) // 32 * 32, "normal")[:, :K].copy()
    wc, ws = amx.quantize(dev_bf16(w_bits), K)
    assert amx.lib().amx_gemm_kernel_for(rows, 70, K, K, amx.GEMM_AUTO) == amx.GEMM_SIMT
    got = amx.gemm(c, s, wc, ws, K).cpu().numpy()
    ref = oracle.gemm(oc, os_, wc.cpu().numpy(), ws.cpu().numpy(), K)
    for m in range(rows):                          # "mixed" rows differ by many orders of magnitude
        if np.all(np.isfinite(ref[m])) and np.linalg.norm(ref[m]) > 0:
            assert rel_fro(got[m], ref[m]) <= 1e-5


def test_config1_both_operands_cast_in_one_call():
    """Config 1 through one call of amx_quant_gemm with the bf16 weight: activation and weight are both cast per
    call; every kernel choice against the oracle, and bit-identical to the cast-then-multiply sequence."""
    a_bits, w_bits = inputs.activation(1, 0), inputs.weight(1, 0)
    a, w = dev_bf16(a_bits), dev_bf16(w_bits)
    qa, qw = oracle.quantize(a_bits, 32), oracle.quantize(w_bits, 32)
    ref = oracle.gemm(*qa, *qw, 32)
    wc, ws = amx.quantize(w, 32)
    for flags in (amx.GEMM_AUTO, amx.GEMM_TC, amx.GEMM_FP4, amx.GEMM_SIMT, amx.GEMM_TC | amx.GEMM_CAST_IN_KERNEL):
        got = amx.quant_gemm(a, flags=flags, w_bf16=w)
        assert rel_fro(got.cpu().numpy(), ref) <= 1e-3, flags
        assert torch.equal(got, amx.quant_gemm(a, wc, ws, 32, flags)), flags
    got16 = amx.quant_gemm(a[:16].contiguous(), flags=amx.GEMM_ROWS, w_bf16=w)
    assert rel_fro(got16.cpu().numpy(), ref[:16]) <= 1e-5
    # row-strided operands (views into wider buffers) take the two-launch route of the FP4 path
    wa = torch.zeros((128, 1024 + 64), dtype=torch.bfloat16, device="cuda")
    ww = torch.zeros((1024, 1024 + 8), dtype=torch.bfloat16, device="cuda")
    wa[:, 8:8 + 1024], ww[:, :1024] = a, w
    got = amx.quant_gemm(wa[:, 8:8 + 1024], flags=amx.GEMM_FP4, w_bf16=ww[:, :1024])
    assert torch.equal(got, amx.quant_gemm(a, flags=amx.GEMM_FP4, w_bf16=w))


def test_both_operands_cast_in_one_call_large_layer():
    """A layer large enough for AUTO to pick the FP4 kernel (config 2, 512 token rows x 4096 -> 4096)."""
    a_bits, w_bits = inputs.activation(2, 1, M=512), inputs.weight(2, 1)
    assert amx.lib().amx_gemm_kernel_for(512, 4096, 4096, 32, 0) == amx.GEMM_FP4
    got = amx.quant_gemm(dev_bf16(a_bits), w_bf16=dev_bf16(w_bits)).cpu().numpy()
    rows = np.arange(0, 512, 8)
    ref = oracle.gemm(*oracle.quantize(a_bits, 32), *oracle.quantize(w_bits, 32), 32, rows=rows)
    assert rel_fro(got[rows], ref) <= 1e-3


@pytest.mark.parametrize("M,flags", [(16, amx.GEMM_AUTO), (16, amx.GEMM_ROWS), (128, amx.GEMM_TC), (128, amx.GEMM_FP4),
                                     (128, amx.GEMM_SIMT)])
def test_status_word_after_every_kernel(M, flags):
    """amx_gemm_status on the workspace of amx_gemm and of amx_quant_gemm: AMX_OK whichever kernel ran, also with a
    workspace that was full of ones before the call."""
    N, K = 512, 1024
    a_bits, w_bits = inputs.random_groups(1900, M, K, "normal"), inputs.random_groups(1901, N, K, "normal")
    a, w = dev_bf16(a_bits), dev_bf16(w_bits)
    (ac, as_), (wc, ws) = amx.quantize(a, 32), amx.quantize(w, 32)
    L = amx.lib()
    work = torch.full((max(256, L.amx_workspace_bytes(M, N, K, 32, flags)),), 0xFF, dtype=torch.uint8, device="cuda")
    amx.gemm(ac, as_, wc, ws, 32, flags, workspace=work)
    if L.amx_workspace_bytes(M, N, K, 32, flags):
        assert amx.gemm_status(work) == 0 and amx.gemm_flushed_scales(work) == 0
    work = torch.full((L.amx_quant_gemm_workspace_bytes(M, N, K, 32, flags),), 0xFF, dtype=torch.uint8, device="cuda")
    amx.quant_gemm(a, wc, ws, 32, flags, workspace=work)
    assert amx.gemm_status(work) == 0 and amx.gemm_flushed_scales(work) == 0


def test_auto_with_two_byte_aligned_weight_scales_for_few_rows():
    """AUTO picks the weight-streaming kernel for 16 rows; that kernel wants 4-byte aligned scales.  A weight whose
    scales are only 2-byte aligned is still multiplied (by the plain kernel) instead of being refused."""
    M, N, K = 16, 256, 1024
    a_bits, w_bits = inputs.random_groups(1910, M, K, "normal"), inputs.random_groups(1911, N, K, "normal")
    qa, qw = oracle.quantize(a_bits, 32), oracle.quantize(w_bits, 32)
    ac, as_, wc = (torch.from_numpy(t).cuda() for t in (qa[0], qa[1], qw[0]))
    buf = torch.zeros(qw[1].size + 2, dtype=torch.uint8, device="cuda")
    buf[2:] = torch.from_numpy(qw[1]).cuda().reshape(-1)
    ws_view = buf[2:].view(N, K // 32, 2)
    assert ws_view.data_ptr() % 4 == 2
    out = torch.empty((M, N), dtype=torch.float32, device="cuda")
    L = amx.lib()
    work = torch.empty(L.amx_workspace_bytes(M, N, K, 32, 0), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    rc = L.amx_gemm(ac.data_ptr(), as_.data_ptr(), wc.data_ptr(), ws_view.data_ptr(), M, N, K, 32, 0, out.data_ptr(), N,
                    work.data_ptr(), work.numel(), stream)
    assert rc == 0
    assert rel_fro(out.cpu().numpy(), oracle.gemm(*qa, *qw, 32)) <= 1e-5
    rc = L.amx_gemm(ac.data_ptr(), as_.data_ptr(), wc.data_ptr(), ws_view.data_ptr(), M, N, K, 32, amx.GEMM_ROWS,
                    out.data_ptr(), N, work.data_ptr(), work.numel(), stream)
    assert rc == -3                                # asked for explicitly: the alignment error stands


def test_bounded_wait_runs_out_and_the_context_survives():
    """A wait on a barrier nothing arrives at gives up after its poll limit: AMX_ERR_TIMEOUT in the status word,
    the waiting role gave up by itself, the others left through the abort flag, the copy in flight was drained;
    afterwards the same context runs a tensor-core GEMM (tensor memory was released) with a clean status."""
    L = amx.lib()
    work = torch.full((4096,), 0xFF, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    assert L.amx_selftest_wait_timeout(work.data_ptr(), work.numel(), 512, stream) == 0
    assert amx.gemm_status(work) == -8 and amx.status_string(-8) == "device-side wait timed out"
    trace = work.view(torch.int32)[8:13].cpu().tolist()
    assert trace == [2, 3, 3, 3, 1], trace
    a_bits, w_bits = inputs.random_groups(1920, 256, 512, "normal"), inputs.random_groups(1921, 512, 512, "normal")
    qa, qw = oracle.quantize(a_bits, 32), oracle.quantize(w_bits, 32)
    dev = [torch.from_numpy(t).cuda() for t in (*qa, *qw)]
    for flags in (amx.GEMM_FP4, amx.GEMM_TC):
        ws = torch.empty(L.amx_workspace_bytes(256, 512, 512, 32, flags), dtype=torch.uint8, device="cuda")
        got = amx.gemm(*dev, 32, flags, workspace=ws)
        assert amx.gemm_status(ws) == 0
        assert rel_fro(got.cpu().numpy(), oracle.gemm(*qa, *qw, 32)) <= 1e-4


@pytest.mark.parametrize("flags", [amx.GEMM_AUTO, amx.GEMM_FP4, amx.GEMM_TC, amx.GEMM_SIMT])
def test_linear_host_with_explicit_kernel(flags):
    """The host-buffer layer sizes its scratch for the kernel that is asked for; two calls without synchronisation
    on two streams give the same results as synchronous ones."""
    M, N, K = 128, 256, 1024
    a_bits, w_bits = inputs.activation(1, 0), inputs.weight(1, 0, N=N)
    a = torch.from_numpy(a_bits.view(np.int16)).view(torch.bfloat16).pin_memory()
    w = torch.from_numpy(w_bits.view(np.int16)).view(torch.bfloat16).pin_memory()
    ref = oracle.gemm(*oracle.quantize(a_bits, 32), *oracle.quantize(w_bits, 32), 32)
    L = amx.lib()
    nbytes = L.amx_linear_host_workspace_bytes(M, N, K, 32, flags)
    c = torch.empty((M, N), dtype=torch.float32).pin_memory()
    amx.linear_host(a, w, c, torch.empty(nbytes, dtype=torch.uint8, device="cuda"), flags=flags)
    assert rel_fro(c.numpy(), ref) <= 1e-3
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = [torch.zeros((M, N), dtype=torch.float32).pin_memory() for _ in streams]
    works = [torch.empty(nbytes, dtype=torch.uint8, device="cuda") for _ in streams]
    torch.cuda.synchronize()
    for st, o, wk in zip(streams, outs, works):
        with torch.cuda.stream(st):
            amx.linear_host(a, w, o, wk, flags=flags | amx.HOST_NO_SYNC)
    torch.cuda.synchronize()
    for o in outs:
        assert np.array_equal(o.numpy(), c.numpy())


@pytest.mark.parametrize("flags", [amx.GEMM_AUTO, amx.GEMM_FP4, amx.GEMM_TC, amx.GEMM_SIMT])
@pytest.mark.parametrize("M,N,K", [(128, 256, 1024), (4500, 520, 1056), (2049, 300, 512), (16, 512, 1024)])
def test_linear_host_pipelined(flags, M, N, K):
    """The three-stream pipeline over row chunks (4500 rows: three chunks of 1536, 1536 and 1428; 2049: 1152 + 897)
    against the oracle and against the one-stream entry point; two layers in flight on the same streams."""
    if not amx.lib().amx_gemm_kernel_for(M, N, K, 32, flags) or not amx.lib().amx_gemm_kernel_for(min(M, 897), N, K, 32, flags):
        pytest.skip("kernel choice does not take this shape")
    a_bits = inputs.random_groups(5100 + M, M, K, "normal")
    w_bits = inputs.random_groups(5200 + N, N, K, "normal")
    a = torch.from_numpy(a_bits.view(np.int16)).view(torch.bfloat16).pin_memory()
    w = torch.from_numpy(w_bits.view(np.int16)).view(torch.bfloat16).pin_memory()
    L = amx.lib()
    nbytes = L.amx_linear_host_pipelined_workspace_bytes(M, N, K, 32, flags)
    assert nbytes > 0
    streams = [torch.cuda.Stream() for _ in range(3)]
    works = [torch.full((nbytes,), 0xFF, dtype=torch.uint8, device="cuda") for _ in range(2)]
    outs = [torch.full((M, N), float("nan"), dtype=torch.float32).pin_memory() for _ in range(2)]
    torch.cuda.synchronize()
    amx.linear_host_pipelined(a, w, outs[0], works[0], streams, flags=flags)                 # synchronous form
    assert L.amx_linear_host_pipelined_status(works[0].data_ptr(), streams[1].cuda_stream) == 0
    ref = oracle.gemm(*oracle.quantize(a_bits, 32), *oracle.quantize(w_bits, 32), 32)
    assert rel_fro(outs[0].numpy(), ref) <= 1e-3
    one = torch.empty((M, N), dtype=torch.float32).pin_memory()
    amx.linear_host(a, w, one, torch.empty(L.amx_linear_host_workspace_bytes(M, N, K, 32, flags), dtype=torch.uint8,
                                           device="cuda"), flags=flags)
    assert rel_fro(outs[0].numpy(), one.numpy().astype(np.float64)) <= 1e-5
    # two calls in flight on the same three streams, a workspace each
    first = outs[0].numpy().copy()
    for o in outs:
        o.fill_(float("nan"))
    for o, wk in zip(outs, works):
        amx.linear_host_pipelined(a, w, o, wk, streams, flags=flags | amx.HOST_NO_SYNC)
    torch.cuda.synchronize()
    for o, wk in zip(outs, works):
        assert np.array_equal(o.numpy(), first)
        assert L.amx_linear_host_pipelined_status(wk.data_ptr(), None) == 0


def test_linear_host_pipelined_argument_errors():
    L = amx.lib()
    a = torch.zeros((128, 64), dtype=torch.bfloat16).pin_memory()
    c = torch.zeros((128, 128), dtype=torch.float32).pin_memory()
    need = L.amx_linear_host_pipelined_workspace_bytes(128, 128, 64, 32, 0)
    ws = torch.empty(need + 256, dtype=torch.uint8, device="cuda")
    streams = [torch.cuda.Stream() for _ in range(3)]
    s = [t.cuda_stream for t in streams]
    args = (a.data_ptr(), a.data_ptr(), 128, 128, 64, 32)
    assert L.amx_linear_host_pipelined(*args, 0, c.data_ptr(), ws.data_ptr(), ws.numel(), s[0], s[0], s[2]) == -5
    assert L.amx_linear_host_pipelined(*args, 0x30, c.data_ptr(), ws.data_ptr(), ws.numel(), *s) == -5
    assert L.amx_linear_host_pipelined(*args, 0, c.data_ptr(), ws.data_ptr(), 1024, *s) == -4
    assert L.amx_linear_host_pipelined(*args, 0, None, ws.data_ptr(), ws.numel(), *s) == -1
    assert L.amx_linear_host_pipelined(a.data_ptr(), a.data_ptr(), 128, 128, 48, 32, 0, c.data_ptr(), ws.data_ptr(), ws.numel(), *s) == -2
    assert L.amx_linear_host_pipelined(*args, 0, c.data_ptr(), ws.data_ptr() + 16, need, *s) == -3
    assert L.amx_linear_host_pipelined_workspace_bytes(128, 128, 48, 32, 0) == 0
    torch.cuda.synchronize()


@pytest.mark.parametrize("rows,K,is_w", [(300, 1056, False), (130, 96, True), (77, 11008, False), (9, 36864, True), (2100, 128, True)])
def test_quantize_prepared_without_canonical_codes(rows, K, is_w):
    """The prepared cast with codes = NULL writes the same scales and the same prepared operand, byte for byte
    (row lengths below, at and above a warp's 32 groups, and beyond the 32 groups per lane held in registers)."""
    bits = inputs.random_groups(2000 + rows, rows, K, "mixed")
    x = dev_bf16(bits)
    nbytes = amx.lib().amx_prepared_bytes(rows, K, 32, int(is_w))
    c, s1, p1 = amx.quantize_prepared(x, is_w, prepared=torch.zeros(nbytes, dtype=torch.uint8, device="cuda"))
    none, s2, p2 = amx.quantize_prepared(x, is_w, prepared=torch.zeros(nbytes, dtype=torch.uint8, device="cuda"),
                                         want_codes=False)
    assert none is None and torch.equal(s1, s2) and torch.equal(p1, p2)
    oc, os_ = oracle.quantize(bits, 32)
    assert np.array_equal(c.cpu().numpy(), oc) and np.array_equal(s1.cpu().numpy(), os_)
    # the positive and negative planes together are the codes
    plane = -(-(rows * K // 2) // 256) * 256
    planes = p1.cpu().numpy()
    assert np.array_equal(planes[: rows * K // 2] | planes[plane: plane + rows * K // 2], oc.reshape(-1))


@pytest.mark.parametrize("fmt", [0, 1, 2, 3, 4, 5])
@pytest.mark.parametrize("gs", [16, 32, 64, 128])
def test_fake_quantize_equals_cast_then_decode(fmt, gs):
    """amx_fake_quantize against the oracle's quantize -> dequantize (every format and group size; ragged row count,
    row-strided input, in place), and against Algorithm 1's own fake-quant routine for MXFP4."""
    rows, K = 77, 5 * 128
    bits = inputs.random_groups(5100 + fmt * 10 + gs, rows, K, "mixed")
    oc, os_ = oracle.quantize(bits, gs) if fmt == 0 else oracle.quantize_variant(bits, gs, fmt)
    want = inputs.f32_to_bf16_bits(oracle.dequantize(oc, os_, gs).astype(np.float32))
    x = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    got = amx.fake_quantize(x, gs, fmt).view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(got, want)
    wide = torch.zeros((rows, K + 24), dtype=torch.bfloat16, device="cuda")
    wide[:, 8:8 + K] = x
    view = wide[:, 8:8 + K]
    amx.fake_quantize(view, gs, fmt, out=view)                        # strided, in place
    assert np.array_equal(view.contiguous().view(torch.int16).cpu().numpy().view(np.uint16), want)
    assert not wide[:, :8].any() and not wide[:, 8 + K:].any()
    if fmt == amx.FMT_MXFP4:
        v = inputs.bf16_bits_to_f32(bits).astype(np.float64)
        keep = np.isfinite(v).all(axis=1)
        alg1 = oracle.fakequant_pot_floor(v[keep], gs, False)
        scale_ok = np.abs(v[keep]).reshape(keep.sum(), -1, gs).max(axis=2)     # inside the E5M2 range of the stored power of two
        inr = np.repeat((scale_ok == 0) | ((scale_ok >= 2.0 ** -14) & (scale_ok < 2.0 ** 17)), gs, axis=1)
        assert np.array_equal(inputs.bf16_bits_to_f32(got[keep]).astype(np.float64)[inr], alg1[inr])
