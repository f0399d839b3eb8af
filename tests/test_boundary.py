"""CPU-side checks of the C-ABI boundary: the library loads without a GPU, exports every symbol the
header declares, and rejects bad arguments on the host before anything is launched."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2411_09909_b200 import build, amx
    build.build()
    return amx.lib()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "amx.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(amx_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    from paper_2411_09909_b200 import amx
    declared = _declared_symbols()
    assert len(declared) >= 13
    for name in declared:
        assert hasattr(L, name), name
    assert sorted(amx.SYMBOLS) == declared


def test_status_strings(L):
    assert L.amx_status_string(0) == b"ok"
    seen = {L.amx_status_string(c) for c in range(-9, 1)}
    assert len(seen) == 10 and b"unknown status" not in seen
    assert L.amx_status_string(-99) == b"unknown status"


def test_host_detected_argument_errors(L):
    fake = ctypes.c_void_p(0x1000)          # never dereferenced: every call below fails validation first
    odd = ctypes.c_void_p(0x1001)
    q = L.amx_quantize
    assert q(None, 0, 64, 64, 32, None, None, None) == 0                # rows == 0: no-op
    assert q(None, 4, 64, 64, 32, None, None, None) == -1               # NULL
    assert q(fake, 4, 64, 64, 24, fake, fake, None) == -2               # group size
    assert q(fake, 4, 80, 80, 32, fake, fake, None) == -2               # K % gs
    assert q(fake, 4, 64, 32, 32, fake, fake, None) == -2               # ld < K
    assert q(odd, 4, 64, 64, 32, fake, fake, None) == -3                # alignment
    assert q(fake, 4, 64, 68, 32, fake, fake, None) == -3               # ld % 8
    assert L.amx_quantize_fmt(fake, 4, 64, 64, 32, 6, fake, fake, None) == -5       # unknown format
    assert L.amx_quantize_fmt(fake, 4, 64, 64, 24, 1, fake, fake, None) == -2
    assert L.amx_quantize_prepared_fmt(fake, 4, 64, 32, 0, 7, fake, fake, fake, 1 << 20, None) == -5
    assert L.amx_quantize_t(fake, 48, 8, 8, 32, fake, fake, None) == -2  # R % gs
    assert L.amx_dequantize(fake, fake, 4, 64, 32, 0x2, fake, 64, None) == -5
    assert L.amx_dequantize(fake, fake, 4, 64, 32, 0, None, 64, None) == -1
    g = L.amx_gemm
    assert g(fake, fake, fake, fake, 4, 4, 64, 32, 0x30, fake, 4, None, 0, None) == -5  # both kernels asked
    assert g(fake, fake, fake, fake, 4, 4, 64, 32, 0x200, fake, 4, None, 0, None) == -5
    assert g(fake, fake, fake, fake, 4, 8, 64, 32, 0, fake, 4, None, 0, None) == -2     # ld_c < N
    assert g(None, fake, fake, fake, 4, 4, 64, 32, 0x10, fake, 4, None, 0, None) == -1
    assert g(fake, fake, fake, fake, 4, 4, 64, 32, 0x100, fake, 4, None, 0, None) == -2     # streaming kernel: K % 128
    assert g(fake, fake, fake, fake, 65, 4, 512, 32, 0x100, fake, 4, None, 0, None) == -2   # and at most 64 rows
    assert g(fake, fake, fake, ctypes.c_void_p(0x1002), 4, 4, 512, 32, 0x100, fake, 4, fake, 1 << 20, None) == -3
    assert g(fake, fake, fake, fake, 0, 4, 64, 32, 0x10, fake, 4, None, 0, None) == 0   # empty
    qg = L.amx_quant_gemm
    assert qg(fake, 64, fake, fake, None, 0, 4, 4, 64, 32, 0x10, fake, 4, None, 0, None) == -4
    assert qg(fake, 64, fake, fake, None, 0, 4, 4, 64, 32, 0x80, fake, 4, fake, 4096, None) == -5   # cast-in-kernel
    assert qg(fake, 64, fake, fake, None, 0, 4, 4, 64, 32, 0xC0, fake, 4, fake, 4096, None) == -5   # needs the TC kernel
    assert qg(fake, 64, fake, fake, fake, 64, 4, 4, 64, 32, 0x10, fake, 4, fake, 1 << 20, None) == -1   # both weight forms
    assert qg(fake, 64, None, None, None, 0, 4, 4, 64, 32, 0x10, fake, 4, fake, 1 << 20, None) == -1    # no weight at all
    assert qg(fake, 64, None, None, fake, 32, 4, 4, 64, 32, 0x10, fake, 4, fake, 1 << 20, None) == -2   # ld_w < K
    assert qg(fake, 64, None, None, odd, 64, 4, 4, 64, 32, 0x10, fake, 4, fake, 1 << 20, None) == -3    # bf16 weight alignment
    assert L.amx_linear_host(fake, fake, 4, 4, 64, 32, 0x30, fake, fake, 1 << 30, None) == -5             # two kernels
    assert L.amx_linear_host(fake, fake, 4, 4, 64, 32, 0x40, fake, fake, 16, None) == -4                  # checked before any copy
    s1, s2, s3 = ctypes.c_void_p(0x100), ctypes.c_void_p(0x200), ctypes.c_void_p(0x300)          # never dereferenced here
    lp = L.amx_linear_host_pipelined
    assert lp(fake, fake, 4, 4, 64, 32, 0x30, fake, fake, 1 << 30, s1, s2, s3) == -5                      # two kernels
    assert lp(fake, fake, 4, 4, 64, 32, 0, fake, fake, 1 << 30, s1, s1, s3) == -5                         # two equal streams
    assert lp(fake, fake, 4, 4, 64, 32, 0, fake, fake, 16, s1, s2, s3) == -4                              # before any copy
    assert lp(fake, fake, 4, 4, 48, 32, 0, fake, fake, 1 << 30, s1, s2, s3) == -2
    assert lp(None, fake, 4, 4, 64, 32, 0, fake, fake, 1 << 30, s1, s2, s3) == -1
    assert L.amx_linear_host_pipelined_workspace_bytes(4096, 256, 512, 32, 0) > L.amx_linear_host_workspace_bytes(2048, 256, 512, 32, 0)
    am = L.amx_attention_map
    assert am(fake, fake, fake, 320, 128, 0, fake, fake, fake, fake, fake, 1 << 30, fake, 1 << 30, None) == -2   # L % 128
    assert am(fake, fake, fake, 512, 64, 0, fake, fake, fake, fake, fake, 1 << 30, fake, 1 << 30, None) == -2    # d != 128
    assert am(fake, fake, fake, 512, 128, 0x40, fake, fake, fake, fake, fake, 1 << 30, fake, 1 << 30, None) == -5
    assert am(fake, fake, None, 512, 128, 0, fake, fake, fake, fake, fake, 1 << 30, fake, 1 << 30, None) == -1
    assert L.amx_prepared_flushed_scales(None, 4, 64, 32, 0, None) == -1
    assert L.amx_prepared_flushed_scales(fake, 4, 64, 16, 0, None) == -2
    assert L.amx_selftest_wait_timeout(fake, 64, 100, None) == -4
    assert L.amx_selftest_wait_timeout(fake, 4096, 0, None) == -2
    # whole-row groups (group_size == K) on the generic entry points; not on the transposed cast
    assert q(fake, 4, 72, 72, 72, None, fake, None) == -1
    assert q(fake, 4, 76, 76, 76, fake, fake, None) == -2               # K % 8
    assert L.amx_dequantize(fake, fake, 4, 72, 72, 0, None, 72, None) == -1
    assert L.amx_gemm_kernel_for(4, 4, 72, 72, 0) == 0x10
    assert L.amx_quantize_t(fake, 48, 8, 8, 48, fake, fake, None) == -2
    assert L.amx_gemm(fake, fake, fake, fake, 4, 4, 64, 32, 0xA0, fake, 4, None, 0, None) == -5          # not an amx_gemm flag
    assert L.amx_attention(fake, fake, fake, 1, 64, 64, 0x2000, fake, fake, 1 << 30, None) == -5           # unknown flag
    assert L.amx_attention(fake, fake, fake, 1, 48, 64, 0x1000, fake, fake, 1 << 30, None) == -2           # L % 32
    assert L.amx_softmax_bf16(fake, 4, 0, 0, 1.0, fake, 0, None) == -2
    assert L.amx_softmax_quantize(fake, 4, 48, 48, ctypes.c_float(1.0), fake, fake, 0, None, 0, None) == -2   # cols % 32
    assert L.amx_softmax_quantize(fake, 4, 64, 32, ctypes.c_float(1.0), fake, fake, 0, None, 0, None) == -2   # ld < cols
    assert L.amx_softmax_quantize(fake, 4, 64, 64, ctypes.c_float(1.0), None, fake, 0, None, 0, None) == -1
    assert L.amx_softmax_quantize(fake, 4, 64, 64, ctypes.c_float(1.0), fake, fake, 0, fake, 16, None) == -4  # prepared too small


def test_workspace_sizes(L):
    assert L.amx_workspace_bytes(128, 128, 100, 32, 0) == 0            # invalid shape
    simt = L.amx_workspace_bytes(100, 100, 64, 32, 0x10)
    assert simt == 0
    qg = L.amx_quant_gemm_workspace_bytes(100, 100, 64, 32, 0x10)
    assert qg >= 100 * 32 + 100 * 2 * 2 and qg % 256 == 0
    assert L.amx_quant_gemm_workspace_bytes(100, 100, 64, 32, 0x10 | 0x200) >= qg + 100 * 32 + 100 * 2 * 2
    lh = L.amx_linear_host_workspace_bytes(128, 256, 512, 32, 0)
    assert lh >= 128 * 512 * 2 + 256 * 512 * 2 + 128 * 256 * 4
    # an explicit kernel choice sizes the scratch for that kernel
    assert L.amx_linear_host_workspace_bytes(128, 256, 512, 32, 0x40) > lh
    # AUTO on the FP4 kernel carries the exact kernel's scratch too (device-side fallback)
    assert L.amx_workspace_bytes(2048, 4096, 4096, 32, 0) > L.amx_workspace_bytes(2048, 4096, 4096, 32, 0x40)
    # the weight-streaming kernel's scratch starts with a status header
    assert L.amx_workspace_bytes(16, 4096, 4096, 32, 0x100) == 256 + 16 * 4096 * 2
    assert L.amx_gemm_kernel_for(100, 100, 64, 32, 0x10) == 0x10


def test_binding_fails_loudly_without_library(monkeypatch, tmp_path):
    from paper_2411_09909_b200 import amx
    monkeypatch.setattr(amx, "_lib", None)
    monkeypatch.setattr(amx, "_LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(amx.AmxError):
        amx.lib()
