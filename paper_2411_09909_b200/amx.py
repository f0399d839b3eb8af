"""Thin Python binding of the C-ABI CUDA library (``include/amx.h``).

Argument marshalling only: every function checks tensor types, allocates outputs with
torch (device memory and streams are all torch is used for) and forwards pointers to the
entry point of the same name.  There is no fallback of any kind: if ``libamx_b200.so``
has not been built (``python -m paper_2411_09909_b200.build``) the first call raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libamx_b200.so")
_lib = None

OUT_BF16, OUT_F32 = 0x0, 0x1
GEMM_AUTO, GEMM_SIMT, GEMM_TC, GEMM_FP4 = 0x0, 0x10, 0x20, 0x40
GEMM_ROWS = 0x100               # weight-streaming kernel for at most 64 rows of A
GEMM_CAST_IN_KERNEL = 0x80      # amx_quant_gemm only, together with GEMM_TC
FMT_AMXFP4, FMT_SYM_FP8, FMT_MXFP4 = 0, 1, 2
FMT_AMXFP4_POT, FMT_MXFP4_POT_ROUND, FMT_AMXFP4_POT_ROUND = 3, 4, 5   # amx_quantize_fmt only
WEIGHT_BF16 = 0x200             # amx_quant_gemm_workspace_bytes: size for a bf16 weight
ATTN_CAUSAL = 0x1000            # amx_attention / amx_attention_map
HOST_NO_SYNC = 0x2000           # amx_linear_host: do not synchronise
PREP_ONE_PLANE, PREP_OUT_BF16 = 0x1, 0x2   # amx_gemm_prepared_ex

# every symbol include/amx.h declares
SYMBOLS = (
    "amx_quantize", "amx_quantize_t", "amx_dequantize", "amx_gemm", "amx_quant_gemm",
    "amx_softmax_bf16", "amx_linear_host", "amx_workspace_bytes",
    "amx_quant_gemm_workspace_bytes", "amx_linear_host_workspace_bytes",
    "amx_gemm_kernel_for", "amx_gemm_status", "amx_status_string",
    "amx_quant_gemm_static", "amx_quant_gemm_static_capacity",
    "amx_attention", "amx_attention_workspace_bytes",
    "amx_prepared_bytes", "amx_prepare", "amx_gemm_prepared", "amx_quantize_prepared", "amx_softmax_quantize",
    "amx_quantize_fmt", "amx_quantize_prepared_fmt", "amx_gemm_prepared_workspace_bytes",
    "amx_quant_error", "amx_quant_error_workspace_bytes",
    "amx_attention_map", "amx_gemm_flushed_scales", "amx_prepared_flushed_scales", "amx_selftest_wait_timeout",
    "amx_quant_gemm_static_status",
    "amx_quantize_nvfp4", "amx_nvfp4_prepared_bytes", "amx_dequantize_nvfp4", "amx_gemm_nvfp4",
    "amx_quantize_f16s", "amx_dequantize_f16s", "amx_gemm_f16s", "amx_quant_error_f16s",
    "amx_fake_quantize", "amx_attention_workspace_bytes_for", "amx_attention_gqa",
    "amx_gemm_prepared_sym", "amx_gemm_nvfp4_sym", "amx_gemm_prepared_ex",
    "amx_linear_host_pipelined", "amx_linear_host_pipelined_workspace_bytes", "amx_linear_host_pipelined_status",
)


class AmxError(RuntimeError):
    pass


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise AmxError(f"{_LIB_PATH} is missing: build it with `python -m paper_2411_09909_b200.build`")
        L = ctypes.CDLL(_LIB_PATH)
        i64, p, i, u32, sz = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_uint32, ctypes.c_size_t
        L.amx_quantize.argtypes = [p, i64, i64, i64, i, p, p, p]
        L.amx_quantize_t.argtypes = [p, i64, i64, i64, i, p, p, p]
        L.amx_quantize_fmt.argtypes = [p, i64, i64, i64, i, i, p, p, p]
        L.amx_quantize_prepared_fmt.argtypes = [p, i64, i64, i, i, i, p, p, p, sz, p]
        L.amx_dequantize.argtypes = [p, p, i64, i64, i, u32, p, i64, p]
        L.amx_gemm.argtypes = [p, p, p, p, i64, i64, i64, i, u32, p, i64, p, sz, p]
        L.amx_quant_error.argtypes = [p, i64, i64, i64, p, p, i, p, p, sz, p]
        L.amx_quant_error_workspace_bytes.argtypes = []
        L.amx_quant_error_workspace_bytes.restype = sz
        L.amx_quant_gemm.argtypes = [p, i64, p, p, p, i64, i64, i64, i64, i, u32, p, i64, p, sz, p]
        L.amx_attention_map.argtypes = [p, p, p, i64, i64, u32, p, p, p, p, p, sz, p, sz, p]
        L.amx_gemm_flushed_scales.argtypes = [p, p]
        L.amx_gemm_flushed_scales.restype = i64
        L.amx_prepared_flushed_scales.argtypes = [p, i64, i64, i, i, p]
        L.amx_prepared_flushed_scales.restype = i64
        L.amx_selftest_wait_timeout.argtypes = [p, sz, u32, p]
        L.amx_quant_gemm_static_status.argtypes = [p]
        L.amx_quantize_nvfp4.argtypes = [p, i64, i64, i64, u32, p, p, p, i, p, sz, p]
        L.amx_nvfp4_prepared_bytes.argtypes = [i64, i64, i]
        L.amx_nvfp4_prepared_bytes.restype = sz
        L.amx_dequantize_nvfp4.argtypes = [p, p, p, i64, i64, u32, p, i64, p]
        L.amx_gemm_nvfp4.argtypes = [p, p, i64, i64, i64, p, i64, p, sz, p]
        L.amx_gemm_nvfp4_sym.argtypes = [p, p, i64, i64, i64, p, i64, p, sz, p]
        L.amx_quantize_f16s.argtypes = [p, i64, i64, i64, i, u32, p, p, p]
        L.amx_fake_quantize.argtypes = [p, i64, i64, i64, i, i, p, i64, p]
        L.amx_dequantize_f16s.argtypes = [p, p, i64, i64, i, p, i64, p]
        L.amx_gemm_f16s.argtypes = [p, p, p, p, i64, i64, i64, i, p, i64, p]
        L.amx_quant_error_f16s.argtypes = [p, i64, i64, i64, p, p, i, p, p, sz, p]
        L.amx_quant_gemm_static.argtypes = [p, i64, p, p, i64, i64, i64, i, u32, p, i64, p]
        L.amx_quant_gemm_static_capacity.argtypes = []
        L.amx_quant_gemm_static_capacity.restype = sz
        L.amx_attention.argtypes = [p, p, p, i64, i64, i64, u32, p, p, sz, p]
        L.amx_attention_gqa.argtypes = [p, p, p, i64, i64, i64, i64, u32, p, p, sz, p]
        L.amx_attention_workspace_bytes.argtypes = [i64, i64]
        L.amx_attention_workspace_bytes.restype = sz
        L.amx_attention_workspace_bytes_for.argtypes = [i64, i64, u32]
        L.amx_attention_workspace_bytes_for.restype = sz
        L.amx_prepared_bytes.argtypes = [i64, i64, i, i]
        L.amx_prepared_bytes.restype = sz
        L.amx_prepare.argtypes = [p, p, i64, i64, i, i, p, sz, p]
        L.amx_quantize_prepared.argtypes = [p, i64, i64, i, i, p, p, p, sz, p]
        L.amx_gemm_prepared.argtypes = [p, p, i64, i64, i64, i, p, i64, p, sz, p]
        L.amx_gemm_prepared_sym.argtypes = [p, p, i64, i64, i64, i, p, i64, p, sz, p]
        L.amx_gemm_prepared_ex.argtypes = [p, p, i64, i64, i64, i, u32, p, i64, p, sz, p]
        L.amx_gemm_prepared_workspace_bytes.argtypes = [i64, i64, i64, i]
        L.amx_gemm_prepared_workspace_bytes.restype = sz
        L.amx_softmax_bf16.argtypes = [p, i64, i64, i64, ctypes.c_float, p, i64, p]
        L.amx_softmax_quantize.argtypes = [p, i64, i64, i64, ctypes.c_float, p, p, i, p, sz, p]
        L.amx_linear_host.argtypes = [p, p, i64, i64, i64, i, u32, p, p, sz, p]
        L.amx_linear_host_pipelined.argtypes = [p, p, i64, i64, i64, i, u32, p, p, sz, p, p, p]
        L.amx_linear_host_pipelined_workspace_bytes.argtypes = [i64, i64, i64, i, u32]
        L.amx_linear_host_pipelined_workspace_bytes.restype = sz
        L.amx_linear_host_pipelined_status.argtypes = [p, p]
        for name in ("amx_workspace_bytes", "amx_quant_gemm_workspace_bytes"):
            getattr(L, name).argtypes = [i64, i64, i64, i, u32]
            getattr(L, name).restype = sz
        L.amx_linear_host_workspace_bytes.argtypes = [i64, i64, i64, i, u32]
        L.amx_linear_host_workspace_bytes.restype = sz
        L.amx_gemm_kernel_for.argtypes = [i64, i64, i64, i, u32]
        L.amx_gemm_kernel_for.restype = u32
        L.amx_gemm_status.argtypes = [p, p]
        L.amx_status_string.argtypes = [i]
        L.amx_status_string.restype = ctypes.c_char_p
        _lib = L
    return _lib


def status_string(rc: int) -> str:
    return lib().amx_status_string(int(rc)).decode()


def _check(rc: int, what: str):
    if rc != 0:
        raise AmxError(f"{what}: {status_string(rc)} ({rc})")


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dev(t: torch.Tensor, dtype, name: str):
    if not t.is_cuda or t.dtype != dtype:
        raise AmxError(f"{name} must be a CUDA tensor of {dtype}")
    return t


def _ws(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def quantize(x: torch.Tensor, group_size: int = 32, fmt: int = FMT_AMXFP4):
    """bf16 [rows, K] (row stride allowed) -> (codes u8 [rows, K/2], scales u8 [rows, K/gs, 2])."""
    _dev(x, torch.bfloat16, "x")
    assert x.dim() == 2 and x.stride(1) == 1
    rows, K = x.shape
    codes = torch.empty((rows, K // 2), dtype=torch.uint8, device=x.device)
    scales = torch.empty((rows, max(K // group_size, 0), 2), dtype=torch.uint8, device=x.device)
    ld = x.stride(0) if rows > 1 else max(K, x.stride(0))
    if fmt == FMT_AMXFP4:
        _check(lib().amx_quantize(x.data_ptr(), rows, K, ld, group_size, codes.data_ptr(), scales.data_ptr(), _stream()),
               "amx_quantize")
    else:
        _check(lib().amx_quantize_fmt(x.data_ptr(), rows, K, ld, group_size, fmt, codes.data_ptr(), scales.data_ptr(),
                                      _stream()), "amx_quantize_fmt")
    return codes, scales


def fake_quantize(x: torch.Tensor, group_size: int = 32, fmt: int = FMT_AMXFP4, out: torch.Tensor | None = None):
    """bf16 [rows, K] (row stride allowed) -> the dequantized cast of x as bf16 (same strides rules); out may be x."""
    _dev(x, torch.bfloat16, "x")
    assert x.dim() == 2 and x.stride(1) == 1
    rows, K = x.shape
    if out is None:
        out = torch.empty((rows, K), dtype=torch.bfloat16, device=x.device)
    assert out.shape == x.shape and out.stride(1) == 1
    ld = lambda t: t.stride(0) if rows > 1 else max(K, t.stride(0))
    _check(lib().amx_fake_quantize(x.data_ptr(), rows, K, ld(x), group_size, fmt, out.data_ptr(), ld(out), _stream()),
           "amx_fake_quantize")
    return out


def quantize_t(x: torch.Tensor, group_size: int = 32):
    """bf16 [R, C], groups down the rows -> canonical quantization of x^T: codes [C, R/2], scales [C, R/gs, 2]."""
    _dev(x, torch.bfloat16, "x")
    assert x.dim() == 2 and x.stride(1) == 1
    R, C = x.shape
    codes = torch.empty((C, R // 2), dtype=torch.uint8, device=x.device)
    scales = torch.empty((C, R // group_size, 2), dtype=torch.uint8, device=x.device)
    _check(lib().amx_quantize_t(x.data_ptr(), R, C, x.stride(0), group_size, codes.data_ptr(),
                                scales.data_ptr(), _stream()), "amx_quantize_t")
    return codes, scales


def dequantize(codes: torch.Tensor, scales: torch.Tensor, group_size: int = 32, dtype=torch.bfloat16):
    _dev(codes, torch.uint8, "codes"), _dev(scales, torch.uint8, "scales")
    rows, K = codes.shape[0], codes.shape[1] * 2
    out = torch.empty((rows, K), dtype=dtype, device=codes.device)
    flag = {torch.bfloat16: OUT_BF16, torch.float32: OUT_F32}[dtype]
    _check(lib().amx_dequantize(codes.data_ptr(), scales.data_ptr(), rows, K, group_size, flag,
                                out.data_ptr(), K, _stream()), "amx_dequantize")
    return out


def quant_error(x: torch.Tensor, codes: torch.Tensor, scales: torch.Tensor, group_size: int = 32) -> torch.Tensor:
    """Device tensor of 4 doubles: sum x^2, sum (x - xhat)^2, its part from clamped elements, their count."""
    _dev(x, torch.bfloat16, "x"), _dev(codes, torch.uint8, "codes"), _dev(scales, torch.uint8, "scales")
    assert x.dim() == 2 and x.stride(1) == 1 and codes.is_contiguous() and scales.is_contiguous()
    rows, K = x.shape
    out = torch.empty(4, dtype=torch.float64, device=x.device)
    ws = torch.empty(lib().amx_quant_error_workspace_bytes(), dtype=torch.uint8, device=x.device)
    _check(lib().amx_quant_error(x.data_ptr(), rows, K, x.stride(0), codes.data_ptr(), scales.data_ptr(), group_size,
                                 out.data_ptr(), ws.data_ptr(), ws.numel(), _stream()), "amx_quant_error")
    return out


def gemm(a_codes, a_scales, w_codes, w_scales, group_size: int = 32, flags: int = GEMM_AUTO,
         out: torch.Tensor | None = None, workspace: torch.Tensor | None = None):
    """fp32 [M, N] = decoded A [M, K] times decoded W [N, K] transposed."""
    for t, n in ((a_codes, "a_codes"), (a_scales, "a_scales"), (w_codes, "w_codes"), (w_scales, "w_scales")):
        _dev(t, torch.uint8, n)
        assert t.is_contiguous()
    M, K = a_codes.shape[0], a_codes.shape[1] * 2
    N = w_codes.shape[0]
    assert w_codes.shape[1] * 2 == K
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32, device=a_codes.device)
    need = lib().amx_workspace_bytes(M, N, K, group_size, flags)
    if workspace is None:
        workspace = _ws(need, a_codes.device)
    _check(lib().amx_gemm(a_codes.data_ptr(), a_scales.data_ptr(), w_codes.data_ptr(), w_scales.data_ptr(),
                          M, N, K, group_size, flags, out.data_ptr(), out.stride(0), workspace.data_ptr(),
                          workspace.numel(), _stream()), "amx_gemm")
    return out


def prepare(codes: torch.Tensor, scales: torch.Tensor, is_weight: bool, group_size: int = 32) -> torch.Tensor:
    """Canonical operand -> prepared operand of the FP4 kernel (reusable across amx_gemm_prepared calls)."""
    _dev(codes, torch.uint8, "codes"), _dev(scales, torch.uint8, "scales")
    rows, K = codes.shape[0], codes.shape[1] * 2
    buf = _ws(lib().amx_prepared_bytes(rows, K, group_size, int(is_weight)), codes.device)
    _check(lib().amx_prepare(codes.data_ptr(), scales.data_ptr(), rows, K, group_size, int(is_weight), buf.data_ptr(),
                             buf.numel(), _stream()), "amx_prepare")
    return buf


def quantize_prepared(x: torch.Tensor, is_weight: bool, group_size: int = 32, prepared: torch.Tensor | None = None,
                      fmt: int = FMT_AMXFP4, want_codes: bool = True):
    """Cast and prepare in one go: returns (codes, scales, prepared); codes is None when want_codes is False."""
    _dev(x, torch.bfloat16, "x")
    assert x.is_contiguous()
    rows, K = x.shape
    codes = torch.empty((rows, K // 2), dtype=torch.uint8, device=x.device) if want_codes else None
    scales = torch.empty((rows, K // group_size, 2), dtype=torch.uint8, device=x.device)
    buf = prepared if prepared is not None else _ws(lib().amx_prepared_bytes(rows, K, group_size, int(is_weight)), x.device)
    if fmt == FMT_AMXFP4:
        _check(lib().amx_quantize_prepared(x.data_ptr(), rows, K, group_size, int(is_weight),
                                           codes.data_ptr() if want_codes else None,
                                           scales.data_ptr(), buf.data_ptr(), buf.numel(), _stream()), "amx_quantize_prepared")
    else:
        _check(lib().amx_quantize_prepared_fmt(x.data_ptr(), rows, K, group_size, int(is_weight), fmt,
                                               codes.data_ptr() if want_codes else None,
                                               scales.data_ptr(), buf.data_ptr(), buf.numel(), _stream()),
               "amx_quantize_prepared_fmt")
    return codes, scales, buf


def gemm_prepared(a_prepared: torch.Tensor, w_prepared: torch.Tensor, M: int, N: int, K: int, group_size: int = 32,
                  out: torch.Tensor | None = None, workspace: torch.Tensor | None = None, sym: bool = False,
                  out_dtype=torch.float32):
    """sym: both operands are in a symmetric format (amx_gemm_prepared_sym; a violated promise shows in gemm_status);
    out_dtype torch.bfloat16: the result rounded to bf16 in the epilogue (amx_gemm_prepared_ex)."""
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=a_prepared.device)
    if workspace is None:
        workspace = _ws(lib().amx_gemm_prepared_workspace_bytes(M, N, K, group_size), a_prepared.device)
    if out.dtype == torch.bfloat16:
        _check(lib().amx_gemm_prepared_ex(a_prepared.data_ptr(), w_prepared.data_ptr(), M, N, K, group_size,
                                          PREP_OUT_BF16 | (PREP_ONE_PLANE if sym else 0), out.data_ptr(), out.stride(0),
                                          workspace.data_ptr(), workspace.numel(), _stream()), "amx_gemm_prepared_ex")
        return out
    _dev(out, torch.float32, "out")
    fn = lib().amx_gemm_prepared_sym if sym else lib().amx_gemm_prepared
    _check(fn(a_prepared.data_ptr(), w_prepared.data_ptr(), M, N, K, group_size, out.data_ptr(),
              out.stride(0), workspace.data_ptr(), workspace.numel(), _stream()), "amx_gemm_prepared")
    return out


def gemm_status(workspace: torch.Tensor) -> int:
    return int(lib().amx_gemm_status(workspace.data_ptr(), _stream()))


def quant_gemm(a: torch.Tensor, w_codes=None, w_scales=None, group_size: int = 32, flags: int = GEMM_AUTO,
               out: torch.Tensor | None = None, workspace: torch.Tensor | None = None, w_bf16: torch.Tensor | None = None):
    """fp32 [M, N] = AMXFP4(a) x W; a is bf16 [M, K]; W is either quantized (w_codes, w_scales) or bf16 [N, K]
    (w_bf16), which the call casts too."""
    _dev(a, torch.bfloat16, "a")
    M, K = a.shape
    if w_bf16 is not None:
        _dev(w_bf16, torch.bfloat16, "w_bf16")
        assert w_codes is None and w_scales is None and w_bf16.stride(1) == 1
    N = w_bf16.shape[0] if w_bf16 is not None else w_codes.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32, device=a.device)
    need = lib().amx_quant_gemm_workspace_bytes(M, N, K, group_size, (flags & ~GEMM_CAST_IN_KERNEL) |
                                                (WEIGHT_BF16 if w_bf16 is not None else 0))
    if workspace is None:
        workspace = _ws(need, a.device)
    _check(lib().amx_quant_gemm(a.data_ptr(), a.stride(0),
                                w_codes.data_ptr() if w_codes is not None else None,
                                w_scales.data_ptr() if w_scales is not None else None,
                                w_bf16.data_ptr() if w_bf16 is not None else None,
                                w_bf16.stride(0) if w_bf16 is not None else 0, M, N, K,
                                group_size, flags, out.data_ptr(), out.stride(0), workspace.data_ptr(),
                                workspace.numel(), _stream()), "amx_quant_gemm")
    return out


def gemm_flushed_scales(workspace: torch.Tensor) -> int:
    return int(lib().amx_gemm_flushed_scales(workspace.data_ptr(), _stream()))


def prepared_flushed_scales(prepared: torch.Tensor, rows: int, K: int, is_weight: bool, group_size: int = 32) -> int:
    return int(lib().amx_prepared_flushed_scales(prepared.data_ptr(), rows, K, group_size, int(is_weight), _stream()))


def attention_map(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, flags: int = 0, want_bf16: bool = True):
    """One head through the attention kernels, with the cast attention map they otherwise never store.
    q, k, v: bf16 [L, 128].  Returns (O fp32 [L, 128], p_bf16 or None, codes, scales, prepared)."""
    for t in (q, k, v):
        _dev(t, torch.bfloat16, "q/k/v")
        assert t.is_contiguous() and t.shape == q.shape
    Lq, d = q.shape
    out = torch.empty((Lq, d), dtype=torch.float32, device=q.device)
    p_bits = torch.empty((Lq, Lq), dtype=torch.bfloat16, device=q.device) if want_bf16 else None
    codes = torch.empty((Lq, Lq // 2), dtype=torch.uint8, device=q.device)
    scales = torch.empty((Lq, Lq // 32, 2), dtype=torch.uint8, device=q.device)
    prep = torch.zeros(max(lib().amx_prepared_bytes(Lq, Lq, 32, 0), 256), dtype=torch.uint8, device=q.device)
    ws = _ws(lib().amx_attention_workspace_bytes(Lq, d), q.device)
    _check(lib().amx_attention_map(q.data_ptr(), k.data_ptr(), v.data_ptr(), Lq, d, flags, out.data_ptr(),
                                   p_bits.data_ptr() if want_bf16 else None, codes.data_ptr(), scales.data_ptr(),
                                   prep.data_ptr(), prep.numel(), ws.data_ptr(), ws.numel(), _stream()), "amx_attention_map")
    return out, p_bits, codes, scales, prep


def softmax_bf16(S: torch.Tensor, alpha: float, out: torch.Tensor | None = None):
    _dev(S, torch.float32, "S")
    rows, cols = S.shape
    if out is None:
        out = torch.empty((rows, cols), dtype=torch.bfloat16, device=S.device)
    _check(lib().amx_softmax_bf16(S.data_ptr(), rows, cols, S.stride(0), float(alpha), out.data_ptr(),
                                  out.stride(0), _stream()), "amx_softmax_bf16")
    return out


def softmax_quantize(S: torch.Tensor, alpha: float, prepared_as: str | None = None):
    """Row softmax, rounding to bf16 and the AMXFP4 cast in one kernel.  Returns (codes, scales) or, with
    prepared_as = "a" / "w", (codes, scales, prepared) for amx_gemm_prepared."""
    _dev(S, torch.float32, "S")
    rows, cols = S.shape
    codes = torch.empty((rows, cols // 2), dtype=torch.uint8, device=S.device)
    scales = torch.empty((rows, cols // 32, 2), dtype=torch.uint8, device=S.device)
    buf, nbytes, is_w = None, 0, int(prepared_as == "w")
    if prepared_as is not None:
        nbytes = lib().amx_prepared_bytes(rows, cols, 32, is_w)
        buf = torch.full((max(nbytes, 256),), 0xFF, dtype=torch.uint8, device=S.device)
    _check(lib().amx_softmax_quantize(S.data_ptr(), rows, cols, S.stride(0), float(alpha), codes.data_ptr(),
                                      scales.data_ptr(), is_w, buf.data_ptr() if buf is not None else None, nbytes,
                                      _stream()), "amx_softmax_quantize")
    return (codes, scales) if buf is None else (codes, scales, buf)


NV_ASYMMETRIC = 0x1


def quantize_nvfp4(x: torch.Tensor, asym: bool, prepared_as: str | None = None):
    """bf16 [rows, K] -> (codes, E4M3 scales [rows, K/16, 2], tensor_scale (2 floats: t, max|x|)[, prepared])."""
    _dev(x, torch.bfloat16, "x")
    assert x.dim() == 2 and x.stride(1) == 1
    rows, K = x.shape
    codes = torch.empty((rows, K // 2), dtype=torch.uint8, device=x.device)
    scales = torch.empty((rows, K // 16, 2), dtype=torch.uint8, device=x.device)
    ts = torch.empty(2, dtype=torch.float32, device=x.device)
    is_w = int(prepared_as == "w")
    prep = None
    if prepared_as is not None:
        prep = torch.full((lib().amx_nvfp4_prepared_bytes(rows, K, is_w),), 0xFF, dtype=torch.uint8, device=x.device)
    _check(lib().amx_quantize_nvfp4(x.data_ptr(), rows, K, x.stride(0), NV_ASYMMETRIC if asym else 0, codes.data_ptr(),
                                    scales.data_ptr(), ts.data_ptr(), is_w, prep.data_ptr() if prep is not None else None,
                                    prep.numel() if prep is not None else 0, _stream()), "amx_quantize_nvfp4")
    return (codes, scales, ts) if prep is None else (codes, scales, ts, prep)


def dequantize_nvfp4(codes: torch.Tensor, scales: torch.Tensor, ts: torch.Tensor, dtype=torch.float32):
    rows, K = codes.shape[0], codes.shape[1] * 2
    out = torch.empty((rows, K), dtype=dtype, device=codes.device)
    flag = {torch.bfloat16: OUT_BF16, torch.float32: OUT_F32}[dtype]
    _check(lib().amx_dequantize_nvfp4(codes.data_ptr(), scales.data_ptr(), ts.data_ptr(), rows, K, flag, out.data_ptr(), K,
                                      _stream()), "amx_dequantize_nvfp4")
    return out


def gemm_nvfp4(a_prepared: torch.Tensor, w_prepared: torch.Tensor, M: int, N: int, K: int, workspace: torch.Tensor | None = None,
               sym: bool = False):
    out = torch.empty((M, N), dtype=torch.float32, device=a_prepared.device)
    if workspace is None:
        workspace = _ws(256, a_prepared.device)
    fn = lib().amx_gemm_nvfp4_sym if sym else lib().amx_gemm_nvfp4
    _check(fn(a_prepared.data_ptr(), w_prepared.data_ptr(), M, N, K, out.data_ptr(), N, workspace.data_ptr(),
              workspace.numel(), _stream()), "amx_gemm_nvfp4")
    return out


F16S_ASYMMETRIC = 0x1
F16S_SCALE_E4M3 = 0x2


def quantize_f16s(x: torch.Tensor, group_size: int = 32, asym: bool = True, e4m3: bool = False):
    """bf16 [rows, K] -> (codes u8 [rows, K/2], binary16 scale bit patterns int16 [rows, K/group_size, 2]);
    e4m3: scales rounded to FP8 E4M3 (stored as the binary16 pattern of that value)."""
    _dev(x, torch.bfloat16, "x")
    assert x.dim() == 2 and x.stride(1) == 1
    rows, K = x.shape
    codes = torch.empty((rows, K // 2), dtype=torch.uint8, device=x.device)
    scales = torch.empty((rows, K // group_size, 2), dtype=torch.int16, device=x.device)
    flags = (F16S_ASYMMETRIC if asym else 0) | (F16S_SCALE_E4M3 if e4m3 else 0)
    _check(lib().amx_quantize_f16s(x.data_ptr(), rows, K, x.stride(0), group_size, flags, codes.data_ptr(), scales.data_ptr(),
                                   _stream()), "amx_quantize_f16s")
    return codes, scales


def dequantize_f16s(codes: torch.Tensor, scales: torch.Tensor, group_size: int = 32) -> torch.Tensor:
    _dev(codes, torch.uint8, "codes"), _dev(scales, torch.int16, "scales")
    assert codes.is_contiguous() and scales.is_contiguous()
    rows, K = codes.shape[0], codes.shape[1] * 2
    out = torch.empty((rows, K), dtype=torch.float32, device=codes.device)
    _check(lib().amx_dequantize_f16s(codes.data_ptr(), scales.data_ptr(), rows, K, group_size, out.data_ptr(), K, _stream()),
           "amx_dequantize_f16s")
    return out


def gemm_f16s(a_codes, a_scales, w_codes, w_scales, group_size: int = 32) -> torch.Tensor:
    for t, d, n in ((a_codes, torch.uint8, "a_codes"), (a_scales, torch.int16, "a_scales"), (w_codes, torch.uint8, "w_codes"),
                    (w_scales, torch.int16, "w_scales")):
        _dev(t, d, n)
        assert t.is_contiguous()
    M, K = a_codes.shape[0], a_codes.shape[1] * 2
    N = w_codes.shape[0]
    assert w_codes.shape[1] * 2 == K
    out = torch.empty((M, N), dtype=torch.float32, device=a_codes.device)
    _check(lib().amx_gemm_f16s(a_codes.data_ptr(), a_scales.data_ptr(), w_codes.data_ptr(), w_scales.data_ptr(), M, N, K,
                               group_size, out.data_ptr(), N, _stream()), "amx_gemm_f16s")
    return out


def quant_error_f16s(x: torch.Tensor, codes: torch.Tensor, scales: torch.Tensor, group_size: int = 32) -> torch.Tensor:
    """quant_error for operands with binary16 scales."""
    _dev(x, torch.bfloat16, "x"), _dev(codes, torch.uint8, "codes"), _dev(scales, torch.int16, "scales")
    assert x.dim() == 2 and x.stride(1) == 1 and codes.is_contiguous() and scales.is_contiguous()
    rows, K = x.shape
    out = torch.empty(4, dtype=torch.float64, device=x.device)
    ws = torch.empty(lib().amx_quant_error_workspace_bytes(), dtype=torch.uint8, device=x.device)
    _check(lib().amx_quant_error_f16s(x.data_ptr(), rows, K, x.stride(0), codes.data_ptr(), scales.data_ptr(), group_size,
                                      out.data_ptr(), ws.data_ptr(), ws.numel(), _stream()), "amx_quant_error_f16s")
    return out


def linear_host(a_host: torch.Tensor, w_host: torch.Tensor, c_host: torch.Tensor, workspace: torch.Tensor,
                group_size: int = 32, flags: int = GEMM_AUTO):
    """Whole layer from (pinned) host bf16 tensors a[M,K], w[N,K] into host fp32 c[M,N]; synchronises unless
    flags carry HOST_NO_SYNC."""
    assert not a_host.is_cuda and not w_host.is_cuda and not c_host.is_cuda and workspace.is_cuda
    assert a_host.dtype == w_host.dtype == torch.bfloat16 and c_host.dtype == torch.float32
    M, K = a_host.shape
    N = w_host.shape[0]
    _check(lib().amx_linear_host(a_host.data_ptr(), w_host.data_ptr(), M, N, K, group_size, flags,
                                 c_host.data_ptr(), workspace.data_ptr(), workspace.numel(), _stream()),
           "amx_linear_host")
    return c_host


def linear_host_pipelined(a_host: torch.Tensor, w_host: torch.Tensor, c_host: torch.Tensor, workspace: torch.Tensor,
                          streams, group_size: int = 32, flags: int = GEMM_AUTO):
    """amx_linear_host as a pipeline over three torch streams (in, compute, out): the rows of a go through in chunks,
    copies in both directions and the kernels overlap.  Synchronises the out stream unless flags carry HOST_NO_SYNC."""
    assert not a_host.is_cuda and not w_host.is_cuda and not c_host.is_cuda and workspace.is_cuda
    assert a_host.dtype == w_host.dtype == torch.bfloat16 and c_host.dtype == torch.float32
    M, K = a_host.shape
    N = w_host.shape[0]
    s_in, s_cmp, s_out = (s.cuda_stream for s in streams)
    _check(lib().amx_linear_host_pipelined(a_host.data_ptr(), w_host.data_ptr(), M, N, K, group_size, flags,
                                           c_host.data_ptr(), workspace.data_ptr(), workspace.numel(), s_in, s_cmp, s_out),
           "amx_linear_host_pipelined")
    return c_host


def attention_heads(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, flags: int = GEMM_AUTO,
                    workspace: torch.Tensor | None = None):
    """Fully quantized attention for all heads through the single C entry point.  q: bf16 [H, L, d]; k, v: bf16
    [H_kv, L, d] with H % H_kv == 0 (grouped queries when H_kv < H); all contiguous.  Returns O fp32 [H, L, d]."""
    for t in (q, k, v):
        _dev(t, torch.bfloat16, "q/k/v")
        assert t.is_contiguous() and t.shape[1:] == q.shape[1:]
    assert k.shape == v.shape
    H, Lq, d = q.shape
    need = lib().amx_attention_workspace_bytes_for(Lq, d, flags)
    if workspace is None:
        workspace = _ws(need, q.device)
    out = torch.empty((H, Lq, d), dtype=torch.float32, device=q.device)
    if k.shape[0] == H:
        _check(lib().amx_attention(q.data_ptr(), k.data_ptr(), v.data_ptr(), H, Lq, d, flags, out.data_ptr(),
                                   workspace.data_ptr(), workspace.numel(), _stream()), "amx_attention")
    else:
        _check(lib().amx_attention_gqa(q.data_ptr(), k.data_ptr(), v.data_ptr(), H, k.shape[0], Lq, d, flags, out.data_ptr(),
                                       workspace.data_ptr(), workspace.numel(), _stream()), "amx_attention_gqa")
    return out


def attention(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, group_size: int = 32, flags: int = GEMM_AUTO):
    """Fully quantized attention for one head (Appendix C: Q, K, the self-attention map and V are all
    quantized): S = AMX(q) AMX(k)^T (groups along head_dim), P = softmax(S / sqrt(d)) rounded to bf16,
    O = AMX(P) AMX(v) with groups along the key axis.  q, k, v: bf16 [L, d].  Returns (O fp32 [L, d], P bf16)."""
    L, d = q.shape
    qc, qs = quantize(q, group_size)
    kc, ks = quantize(k, group_size)
    S = gemm(qc, qs, kc, ks, group_size, flags)
    P = softmax_bf16(S, d ** -0.5)
    pc, ps = quantize(P, group_size)
    vc, vs = quantize_t(v, group_size)
    return gemm(pc, ps, vc, vs, group_size, flags), P
