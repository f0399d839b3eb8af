"""ctypes front end of the AMXFP4 CPU oracle (``amx_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
CPU-baseline leg of the benchmark.  The CUDA library never touches it.

``build()`` compiles the C file with gcc into ``oracle/_build/`` (rebuilt when
the source is newer); every wrapper below marshals numpy arrays and nothing else.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "amx_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_OUT = os.path.join(_OUT_DIR, "libamx_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    os.makedirs(_OUT_DIR, exist_ok=True)
    if force or not os.path.exists(_OUT) or os.path.getmtime(_OUT) < os.path.getmtime(_SRC):
        tmp = _OUT + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
             "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _OUT)
    return _OUT


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i64, dbl, p = ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        L.amx_oracle_e2m1_value.restype = dbl
        L.amx_oracle_e2m1_value.argtypes = [ctypes.c_int]
        L.amx_oracle_e2m1_encode.restype = ctypes.c_int
        L.amx_oracle_e2m1_encode.argtypes = [dbl]
        L.amx_oracle_e5m2_value.restype = dbl
        L.amx_oracle_e5m2_value.argtypes = [ctypes.c_uint8]
        L.amx_oracle_e5m2_encode.restype = ctypes.c_uint8
        L.amx_oracle_e5m2_encode.argtypes = [dbl]
        L.amx_oracle_quantize.argtypes = [p, i64, i64, i64, ctypes.c_int, p, p]
        L.amx_oracle_quantize_variant.argtypes = [p, i64, i64, i64, ctypes.c_int, ctypes.c_int, p, p]
        L.amx_oracle_quantize_f64.argtypes = [p, i64, i64, ctypes.c_int, p, p]
        L.amx_oracle_dequantize.argtypes = [p, p, i64, i64, ctypes.c_int, p]
        L.amx_oracle_gemm.argtypes = [p, p, p, p, i64, i64, i64, ctypes.c_int, p, i64, p]
        L.amx_oracle_quant_error.argtypes = [p, i64, i64, i64, p, p, ctypes.c_int, p]
        L.amx_oracle_fakequant_pot_floor.argtypes = [p, i64, i64, ctypes.c_int, ctypes.c_int, p]
        L.amx_oracle_softmax_bf16.argtypes = [p, i64, i64, dbl, p]
        L.amx_oracle_softmax_bf16_causal.argtypes = [p, i64, i64, dbl, i64, p]
        L.amx_oracle_e4m3_value.restype = dbl
        L.amx_oracle_e4m3_value.argtypes = [ctypes.c_uint8]
        L.amx_oracle_e4m3_encode.restype = ctypes.c_uint8
        L.amx_oracle_e4m3_encode.argtypes = [dbl]
        L.amx_oracle_quantize_nv.argtypes = [p, i64, i64, i64, ctypes.c_int, p, p, p]
        L.amx_oracle_dequantize_nv.argtypes = [p, p, ctypes.c_float, i64, i64, p]
        L.amx_oracle_gemm_nv.argtypes = [p, p, ctypes.c_float, p, p, ctypes.c_float, i64, i64, i64, p, i64, p]
        L.amx_oracle_f16_value.restype = dbl
        L.amx_oracle_f16_value.argtypes = [ctypes.c_uint16]
        L.amx_oracle_f16_encode.restype = ctypes.c_uint16
        L.amx_oracle_f16_encode.argtypes = [dbl]
        L.amx_oracle_quantize_f16s.argtypes = [p, i64, i64, i64, ctypes.c_int, ctypes.c_int, ctypes.c_int, p, p]
        L.amx_oracle_dequantize_f16s.argtypes = [p, p, i64, i64, ctypes.c_int, p]
        L.amx_oracle_gemm_f16s.argtypes = [p, p, p, p, i64, i64, i64, ctypes.c_int, p]
        L.amx_oracle_quant_error_f16s.argtypes = [p, i64, i64, i64, p, p, ctypes.c_int, p]
        L.amx_oracle_num_threads.restype = ctypes.c_int
        _lib = L
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def num_threads() -> int:
    return int(lib().amx_oracle_num_threads())


def e2m1_value(code4: int) -> float:
    return float(lib().amx_oracle_e2m1_value(int(code4)))


def e2m1_encode(r: float) -> int:
    return int(lib().amx_oracle_e2m1_encode(float(r)))


def e5m2_value(code: int) -> float:
    return float(lib().amx_oracle_e5m2_value(int(code)))


def e5m2_encode(q: float) -> int:
    return int(lib().amx_oracle_e5m2_encode(float(q)))


def quantize(x_bf16_bits: np.ndarray, group_size: int = 32):
    """bf16 bit patterns [rows, K] -> (codes u8 [rows, K/2], scales u8 [rows, K/gs, 2])."""
    x = _c(x_bf16_bits, np.uint16)
    rows, K = x.shape
    codes = np.zeros((rows, K // 2), np.uint8)
    scales = np.zeros((rows, K // group_size, 2), np.uint8)
    rc = lib().amx_oracle_quantize(_ptr(x), rows, K, K, group_size, _ptr(codes), _ptr(scales))
    if rc:
        raise ValueError(f"amx_oracle_quantize: bad shape (rc={rc})")
    return codes, scales


SYMMETRIC_FP8, MXFP4 = 1, 2
AMXFP4_POT, MXFP4_POT_ROUND, AMXFP4_POT_ROUND = 3, 4, 5


def quantize_variant(x_bf16_bits: np.ndarray, group_size: int, mode: int):
    """The symmetric comparison formats in AMXFP4's storage layout (both scale bytes equal): mode SYMMETRIC_FP8 =
    one E5M2 scale per group from max|x| / 6; mode MXFP4 = Algorithm 1's power-of-two floor scale.  The per-sign
    power-of-two variants (AMXFP4_POT: floor; *_POT_ROUND: exponent rounded instead of floored, symmetric or
    per sign) use the two bytes like AMXFP4."""
    x = _c(x_bf16_bits, np.uint16)
    rows, K = x.shape
    codes = np.zeros((rows, K // 2), np.uint8)
    scales = np.zeros((rows, K // group_size, 2), np.uint8)
    rc = lib().amx_oracle_quantize_variant(_ptr(x), rows, K, K, group_size, mode, _ptr(codes), _ptr(scales))
    if rc != 0:
        raise ValueError("bad shape, group size or mode")
    return codes, scales


def quantize_f64(x: np.ndarray, group_size: int):
    """fp64 values [rows, K] -> (one 4-bit code per byte [rows, K], scales [rows, K/gs, 2])."""
    x = _c(x, np.float64)
    rows, K = x.shape
    code4 = np.zeros((rows, K), np.uint8)
    scales = np.zeros((rows, K // group_size, 2), np.uint8)
    rc = lib().amx_oracle_quantize_f64(_ptr(x), rows, K, group_size, _ptr(code4), _ptr(scales))
    if rc:
        raise ValueError(f"amx_oracle_quantize_f64: bad shape (rc={rc})")
    return code4, scales


def pack_codes(code4: np.ndarray) -> np.ndarray:
    """One code per byte [rows, K] -> packed [rows, K/2], element 2j in the low nibble."""
    return (code4[:, 0::2] | (code4[:, 1::2] << 4)).astype(np.uint8)


def unpack_codes(codes: np.ndarray) -> np.ndarray:
    out = np.empty((codes.shape[0], codes.shape[1] * 2), np.uint8)
    out[:, 0::2] = codes & 15
    out[:, 1::2] = codes >> 4
    return out


def dequantize(codes: np.ndarray, scales: np.ndarray, group_size: int = 32) -> np.ndarray:
    codes, scales = _c(codes, np.uint8), _c(scales, np.uint8)
    rows, K = codes.shape[0], codes.shape[1] * 2
    out = np.zeros((rows, K), np.float64)
    rc = lib().amx_oracle_dequantize(_ptr(codes), _ptr(scales), rows, K, group_size, _ptr(out))
    if rc:
        raise ValueError(f"amx_oracle_dequantize: bad shape (rc={rc})")
    return out


def quant_error(x_bf16_bits: np.ndarray, codes: np.ndarray, scales: np.ndarray, group_size: int = 32) -> np.ndarray:
    """[sum x^2, sum (x - xhat)^2, its part from clamped elements (|x| > 6 * side scale), their count] in fp64."""
    x, codes, scales = _c(x_bf16_bits, np.uint16), _c(codes, np.uint8), _c(scales, np.uint8)
    rows, K = x.shape
    out = np.zeros(4, np.float64)
    rc = lib().amx_oracle_quant_error(_ptr(x), rows, K, K, _ptr(codes), _ptr(scales), group_size, _ptr(out))
    if rc:
        raise ValueError(f"amx_oracle_quant_error: bad shape (rc={rc})")
    return out


def gemm(codesA, scalesA, codesW, scalesW, group_size: int = 32, rows=None) -> np.ndarray:
    """fp32 [len(rows) or M, N] = decoded A (selected rows) times decoded W transposed, fp64 sums."""
    codesA, scalesA = _c(codesA, np.uint8), _c(scalesA, np.uint8)
    codesW, scalesW = _c(codesW, np.uint8), _c(scalesW, np.uint8)
    M, K = codesA.shape[0], codesA.shape[1] * 2
    N = codesW.shape[0]
    assert codesW.shape[1] * 2 == K
    if rows is None:
        idx, n_rows, idx_p = None, M, None
    else:
        idx = _c(rows, np.int64)
        n_rows, idx_p = idx.shape[0], _ptr(idx)
    C = np.zeros((n_rows, N), np.float32)
    rc = lib().amx_oracle_gemm(_ptr(codesA), _ptr(scalesA), _ptr(codesW), _ptr(scalesW),
                               M, N, K, group_size, idx_p, n_rows, _ptr(C))
    if rc:
        raise ValueError(f"amx_oracle_gemm failed (rc={rc})")
    return C


def fakequant_pot_floor(x: np.ndarray, group_size: int, asym: bool) -> np.ndarray:
    x = _c(x, np.float64)
    rows, K = x.shape
    out = np.zeros_like(x)
    rc = lib().amx_oracle_fakequant_pot_floor(_ptr(x), rows, K, group_size, int(asym), _ptr(out))
    if rc:
        raise ValueError("amx_oracle_fakequant_pot_floor: bad shape")
    return out


def softmax_bf16(S: np.ndarray, alpha: float, causal_row0: int | None = None) -> np.ndarray:
    """Row softmax of alpha*S (fp64), rounded to bf16 bit patterns.  causal_row0: row r is query causal_row0 + r
    and sees columns 0 .. causal_row0 + r only (the rest get 0)."""
    S = _c(S, np.float32)
    rows, cols = S.shape
    P = np.zeros((rows, cols), np.uint16)
    if causal_row0 is None:
        lib().amx_oracle_softmax_bf16(_ptr(S), rows, cols, float(alpha), _ptr(P))
    else:
        lib().amx_oracle_softmax_bf16_causal(_ptr(S), rows, cols, float(alpha), int(causal_row0), _ptr(P))
    return P


# ---- NVFP4 / ANVFP4 (group 16, E4M3 group scales, one fp32 tensor scale) ----

def e4m3_value(code: int) -> float:
    return float(lib().amx_oracle_e4m3_value(int(code)))


def e4m3_encode(q: float) -> int:
    return int(lib().amx_oracle_e4m3_encode(float(q)))


def quantize_nv(x_bf16_bits: np.ndarray, asym: bool):
    """bf16 bit patterns [rows, K] -> (codes u8 [rows, K/2], E4M3 scales u8 [rows, K/16, 2], tensor scale float32).
    asym False: NVFP4 (the group's one scale in both bytes); True: ANVFP4 (positive-side, negative-side scale)."""
    x = _c(x_bf16_bits, np.uint16)
    rows, K = x.shape
    codes = np.zeros((rows, K // 2), np.uint8)
    scales = np.zeros((rows, K // 16, 2), np.uint8)
    t = np.zeros(1, np.float32)
    rc = lib().amx_oracle_quantize_nv(_ptr(x), rows, K, K, int(asym), _ptr(codes), _ptr(scales), _ptr(t))
    if rc:
        raise ValueError("amx_oracle_quantize_nv: K must be a multiple of 16")
    return codes, scales, np.float32(t[0])


def dequantize_nv(codes: np.ndarray, scales: np.ndarray, tensor_scale) -> np.ndarray:
    codes, scales = _c(codes, np.uint8), _c(scales, np.uint8)
    rows, K = codes.shape[0], codes.shape[1] * 2
    out = np.zeros((rows, K), np.float64)
    rc = lib().amx_oracle_dequantize_nv(_ptr(codes), _ptr(scales), float(tensor_scale), rows, K, _ptr(out))
    if rc:
        raise ValueError("amx_oracle_dequantize_nv: bad shape")
    return out


def gemm_nv(codesA, scalesA, tA, codesW, scalesW, tW, rows=None) -> np.ndarray:
    codesA, scalesA = _c(codesA, np.uint8), _c(scalesA, np.uint8)
    codesW, scalesW = _c(codesW, np.uint8), _c(scalesW, np.uint8)
    M, K = codesA.shape[0], codesA.shape[1] * 2
    N = codesW.shape[0]
    assert codesW.shape[1] * 2 == K
    if rows is None:
        idx, n_rows, idx_p = None, M, None
    else:
        idx = _c(rows, np.int64)
        n_rows, idx_p = idx.shape[0], _ptr(idx)
    C = np.zeros((n_rows, N), np.float32)
    rc = lib().amx_oracle_gemm_nv(_ptr(codesA), _ptr(scalesA), float(tA), _ptr(codesW), _ptr(scalesW), float(tW),
                                  M, N, K, idx_p, n_rows, _ptr(C))
    if rc:
        raise ValueError(f"amx_oracle_gemm_nv failed (rc={rc})")
    return C


# ---- FP16 shared scales (the scale-encoding ablation of the appendix) ----

def f16_value(bits: int) -> float:
    return float(lib().amx_oracle_f16_value(int(bits)))


def f16_encode(q: float) -> int:
    return int(lib().amx_oracle_f16_encode(float(q)))


def quantize_f16s(x_bf16_bits: np.ndarray, group_size: int, asym: bool, e4m3: bool = False):
    """bf16 bit patterns [rows, K] -> (codes u8 [rows, K/2], binary16 scales u16 [rows, K/gs, 2]).
    asym True: one scale per sign (positive side, negative side); False: the group's one scale in both.
    e4m3 True: scales rounded to FP8 E4M3 ("1-4-3") and stored as the binary16 pattern of that value."""
    x = _c(x_bf16_bits, np.uint16)
    rows, K = x.shape
    codes = np.zeros((rows, K // 2), np.uint8)
    scales = np.zeros((rows, K // group_size, 2), np.uint16)
    rc = lib().amx_oracle_quantize_f16s(_ptr(x), rows, K, K, int(group_size), int(asym), int(e4m3), _ptr(codes), _ptr(scales))
    if rc:
        raise ValueError("amx_oracle_quantize_f16s: K must be a multiple of the group size")
    return codes, scales


def dequantize_f16s(codes: np.ndarray, scales: np.ndarray, group_size: int) -> np.ndarray:
    codes, scales = _c(codes, np.uint8), _c(scales, np.uint16)
    rows, K = codes.shape[0], codes.shape[1] * 2
    out = np.zeros((rows, K), np.float64)
    rc = lib().amx_oracle_dequantize_f16s(_ptr(codes), _ptr(scales), rows, K, int(group_size), _ptr(out))
    if rc:
        raise ValueError("amx_oracle_dequantize_f16s: bad shape")
    return out


def gemm_f16s(codesA, scalesA, codesW, scalesW, group_size: int) -> np.ndarray:
    codesA, scalesA = _c(codesA, np.uint8), _c(scalesA, np.uint16)
    codesW, scalesW = _c(codesW, np.uint8), _c(scalesW, np.uint16)
    M, K = codesA.shape[0], codesA.shape[1] * 2
    N = codesW.shape[0]
    assert codesW.shape[1] * 2 == K
    C = np.zeros((M, N), np.float32)
    rc = lib().amx_oracle_gemm_f16s(_ptr(codesA), _ptr(scalesA), _ptr(codesW), _ptr(scalesW), M, N, K, int(group_size),
                                    _ptr(C))
    if rc:
        raise ValueError(f"amx_oracle_gemm_f16s failed (rc={rc})")
    return C


def quant_error_f16s(x_bf16_bits: np.ndarray, codes: np.ndarray, scales: np.ndarray, group_size: int) -> np.ndarray:
    x, codes, scales = _c(x_bf16_bits, np.uint16), _c(codes, np.uint8), _c(scales, np.uint16)
    rows, K = x.shape
    out = np.zeros(4, np.float64)
    rc = lib().amx_oracle_quant_error_f16s(_ptr(x), rows, K, K, _ptr(codes), _ptr(scales), int(group_size), _ptr(out))
    if rc:
        raise ValueError("amx_oracle_quant_error_f16s: bad shape")
    return out
