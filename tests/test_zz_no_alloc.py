"""amx_quant_gemm_static: the layer call for callers that cannot allocate device memory (a server
whose own pool owns the whole GPU, a plug-in barred from the allocator, a latency-critical loop).
Its scratch is a fixed array inside the library instead of a caller-provided workspace, so its
result must equal amx_quant_gemm's - also on the second call, when the array still holds the
first call's data.  Collected last on purpose (file name), so that a stop-at-first-failure run
has already exercised everything else."""
import numpy as np
import pytest
import torch

from paper_2411_09909_b200 import amx, inputs

pytestmark = pytest.mark.gpu


def _dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def _static(a, wc, ws, flags=0):
    M, K = a.shape
    N = wc.shape[0]
    out = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    rc = amx.lib().amx_quant_gemm_static(a.data_ptr(), a.stride(0), wc.data_ptr(), ws.data_ptr(), M, N, K, 32,
                                         flags, out.data_ptr(), N, stream)
    assert rc == 0, amx.status_string(rc)
    assert amx.lib().amx_quant_gemm_static_status(stream) == 0       # no bounded wait expired
    return out


def test_static_scratch_entry_point_matches_workspace_entry_point_twice():
    L = amx.lib()
    assert L.amx_quant_gemm_static_capacity() == 16 << 20
    wc, ws = amx.quantize(_dev(inputs.weight(2, 1, N=512)), 32)
    # two different problems back to back: the second must not see anything of the first
    for M, seed_layer in ((384, 0), (200, 1)):
        a = _dev(inputs.activation(2, seed_layer, M=M))
        want = amx.quant_gemm(a, wc, ws, 32)
        got = _static(a, wc, ws)
        torch.cuda.synchronize()
        ref, g = want.double().cpu().numpy(), got.double().cpu().numpy()
        assert np.linalg.norm(g - ref) <= 1e-3 * np.linalg.norm(ref)
        assert torch.equal(got, want)            # same kernels on the same data: identical bits
    # and the SIMT kernel through the same entry point
    a = _dev(inputs.activation(2, 0, M=64))
    assert torch.equal(_static(a, wc, ws, amx.GEMM_SIMT), amx.quant_gemm(a, wc, ws, 32, amx.GEMM_SIMT))


def test_static_scratch_entry_point_rejects_oversized_problems():
    L = amx.lib()
    M, N, K = 16384, 256, 4096                    # quantized activation alone is 36 MiB > 16 MiB
    assert L.amx_quant_gemm_workspace_bytes(M, N, K, 32, 0) > L.amx_quant_gemm_static_capacity()
    a = torch.zeros((8, K), dtype=torch.bfloat16, device="cuda")      # never read: the call is refused first
    dummy = torch.zeros(16, dtype=torch.uint8, device="cuda")
    out = torch.zeros(4, dtype=torch.float32, device="cuda")
    rc = L.amx_quant_gemm_static(a.data_ptr(), K, dummy.data_ptr(), dummy.data_ptr(), M, N, K, 32, 0,
                                 out.data_ptr(), N, None)
    assert rc == -9 and "capacity" in amx.status_string(rc)
