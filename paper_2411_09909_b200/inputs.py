"""Seeded synthetic inputs for the AMXFP4 quantize + GEMM path.

This module only *draws* tensors (numpy Philox, fp32 -> bf16 bit patterns).  It
contains none of the AMXFP4 arithmetic, so the CPU oracle's tests and the CUDA
path can both use it and still share no method code.

The tensors stand in for LLM activations and weights, which the paper evaluates
on real checkpoints that are not available offline.  Their structure follows
what the paper reports about such tensors: a few channels carry outliers that
are tens of times larger than the rest (Section 3.1), groups of 32 have a
non-zero mean (Section 3.1, group-mean discussion), and gated-MLP activations
are skewed (Section 3.1, GLU amplification).

Workloads ("configs"), all generated from ``seed = 24110900 + 100*config +
tensor_index``:

  1  one linear layer, A[128,1024] ~ N(0,1) with 10 channels replaced by
     40*(z+0.5); W[1024,1024] ~ N(0, 0.02)
  2  LLaMA-7B-shaped prefill linears, M=2048: 4096->12288, 4096->4096,
     4096->11008, 11008->4096; A ~ N(0,1) + per-channel offset N(0,0.3),
     0.5 % of the channels x60; W ~ N(0, 0.02)
  3  LLaMA-3-8B-shaped, M=8192: 4096->6144, 4096->14336 (gate), 4096->14336
     (up), 14336->4096; A = SiLU(N(0,1.5)); W ~ N(0, 0.02)
  4  70B-shaped, M=16384: 8192->10240, 8192->28672, 28672->8192; A ~ N(0,1),
     0.2 % of the channels x100; W ~ N(0, 0.01)
  5  attention, 32 heads x 8192 tokens x head_dim 128: Q, K, V ~ N(0,1) with 2
     head-dims x20 per tensor

The second parameter of N(.,.) is the standard deviation.
"""
from __future__ import annotations

import numpy as np

BASE_SEED = 24110900

# (K, N) per layer; M is per config.
LINEAR_CONFIGS = {
    1: {"M": 128, "layers": [(1024, 1024)]},
    2: {"M": 2048, "layers": [(4096, 12288), (4096, 4096), (4096, 11008), (11008, 4096)]},
    3: {"M": 8192, "layers": [(4096, 6144), (4096, 14336), (4096, 14336), (14336, 4096)]},
    4: {"M": 16384, "layers": [(8192, 10240), (8192, 28672), (28672, 8192)]},
}
ATTENTION_CONFIG = {"heads": 32, "seq": 8192, "head_dim": 128}


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even) and return the uint16 bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounding = ((b >> 16) & 1) + np.uint32(0x7FFF)
    return ((b + rounding) >> 16).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32 values."""
    return (bits.astype(np.uint32) << 16).view(np.float32)


def _rng(config: int, tensor_index: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(BASE_SEED + 100 * config + tensor_index))


def _normal(rng, shape, std=1.0):
    x = rng.standard_normal(shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    return x


def activation(config: int, layer: int, M: int | None = None) -> np.ndarray:
    """bf16 bit patterns [M, K] of the activation feeding `layer` of `config` (1..4).

    `M` overrides the number of token rows (rows are i.i.d., so a smaller M is a
    prefix-independent sample of the same distribution).
    """
    spec = LINEAR_CONFIGS[config]
    K, _ = spec["layers"][layer]
    M = spec["M"] if M is None else M
    rng = _rng(config, 2 * layer)
    if config == 1:
        ch = rng.choice(K, size=10, replace=False)
        x = _normal(rng, (M, K))
        x[:, ch] = 40.0 * (x[:, ch] + 0.5)
    elif config == 2:
        mu = _normal(rng, (K,), 0.3)
        ch = rng.choice(K, size=max(1, round(0.005 * K)), replace=False)
        x = _normal(rng, (M, K)) + mu[None, :]
        x[:, ch] *= 60.0
    elif config == 3:
        z = _normal(rng, (M, K), 1.5)
        x = z / (1.0 + np.exp(-z))
    elif config == 4:
        ch = rng.choice(K, size=max(1, round(0.002 * K)), replace=False)
        x = _normal(rng, (M, K))
        x[:, ch] *= 100.0
    else:
        raise ValueError(f"no linear config {config}")
    return f32_to_bf16_bits(x)


def weight(config: int, layer: int, N: int | None = None) -> np.ndarray:
    """bf16 bit patterns [N, K] of the weight of `layer` of `config` (1..4)."""
    spec = LINEAR_CONFIGS[config]
    K, N_full = spec["layers"][layer]
    N = N_full if N is None else N
    std = 0.01 if config == 4 else 0.02
    return f32_to_bf16_bits(_normal(_rng(config, 2 * layer + 1), (N, K), std))


def attention_qkv(heads: int | None = None, seq: int | None = None):
    """bf16 bit patterns of Q, K, V, each [heads, seq, head_dim], for config 5."""
    H = ATTENTION_CONFIG["heads"] if heads is None else heads
    L = ATTENTION_CONFIG["seq"] if seq is None else seq
    D = ATTENTION_CONFIG["head_dim"]
    out = []
    for t in range(3):
        rng = _rng(5, t)
        dims = rng.choice(D, size=2, replace=False)
        x = _normal(rng, (H, L, D))
        x[:, :, dims] *= 20.0
        out.append(f32_to_bf16_bits(x))
    return tuple(out)


def random_groups(seed: int, rows: int, K: int, kind: str = "mixed") -> np.ndarray:
    """Assorted bf16 test rows: wide dynamic range, one-sided groups, zeros, ties.

    kind: "normal"  N(0,1)
          "wide"    N(0,1) * 2^U(-20, 20) per element
          "mixed"   per 32-element block one of: normal, all-positive, all-negative,
                    all-zero, tiny (scale underflow), huge, small-integer/4 grid (many
                    exact rounding ties)
    """
    rng = np.random.Generator(np.random.Philox(BASE_SEED + 7000 + seed))
    x = _normal(rng, (rows, K))
    if kind == "normal":
        return f32_to_bf16_bits(x)
    if kind == "wide":
        x *= np.exp2(rng.integers(-20, 21, size=(rows, K))).astype(np.float32)
        return f32_to_bf16_bits(x)
    assert K % 32 == 0
    g = x.reshape(rows, K // 32, 32)
    sel = rng.integers(0, 8, size=(rows, K // 32))
    g[sel == 1] = np.abs(g[sel == 1])
    g[sel == 2] = -np.abs(g[sel == 2])
    g[sel == 3] = 0.0
    g[sel == 4] *= np.float32(2.0 ** -24)
    g[sel == 5] *= np.float32(2.0 ** 60)
    grid = rng.integers(-24, 25, size=g.shape).astype(np.float32) / 4.0
    g[sel == 6] = grid[sel == 6]
    neg_zero = rng.random(g.shape) < 0.02
    g[neg_zero & (sel == 7)[..., None]] = -0.0
    return f32_to_bf16_bits(g.reshape(rows, K))
