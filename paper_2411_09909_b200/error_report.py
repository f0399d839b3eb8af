"""Synthetic quantization-error report: relative squared error of AMXFP4 and of the symmetric comparison formats
across group sizes, split into the max-clamping and the rounding part (arXiv 2411.09909, appendix "Determining PoT
Shared Scale: Floor vs. Round" and the shared-scale ablation, whose FP16-scale rows come from amx_quantize_f16s
and amx_quant_error_f16s).  Runs on the GPU through amx_quantize(_fmt) and
amx_quant_error on seeded synthetic tensors shaped like the paper's workloads; the paper's own numbers come from
LLM checkpoints and are not reproduced here.

    python -m paper_2411_09909_b200.error_report [--rows 2048]
"""
from __future__ import annotations

import argparse

import numpy as np
import torch

from . import amx, build, inputs

FORMATS = (("AMXFP4 (two FP8 scales)", amx.FMT_AMXFP4), ("symmetric, FP8 scale", amx.FMT_SYM_FP8),
           ("MXFP4 (power-of-two floor)", amx.FMT_MXFP4), ("per-sign power-of-two floor", amx.FMT_AMXFP4_POT),
           ("power-of-two round", amx.FMT_MXFP4_POT_ROUND), ("per-sign power-of-two round", amx.FMT_AMXFP4_POT_ROUND),
           ("symmetric, FP16 scale", "f16s"), ("two FP16 scales", "f16s-asym"),
           ("symmetric, FP8 E4M3 scale", "e4m3"), ("two FP8 E4M3 scales", "e4m3-asym"))
TENSORS = (("activation, channel outliers (config 2, 4096 wide)", 2, 0, "a"),
           ("activation, SiLU-skewed (config 3, 14336 wide)", 3, 3, "a"),
           ("weight N(0, 0.02) (config 2, 4096 -> 4096)", 2, 1, "w"))


def _tensor(config: int, layer: int, kind: str, rows: int) -> torch.Tensor:
    bits = inputs.activation(config, layer, M=rows) if kind == "a" else inputs.weight(config, layer)[:rows]
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def report(rows: int = 2048):
    lines = []
    for title, config, layer, kind in TENSORS:
        x = _tensor(config, layer, kind, rows)
        lines.append(f"\n{title}: {x.shape[0]} x {x.shape[1]}")
        lines.append("| format | group | error / signal | clamping share of the error | elements clamped |")
        lines.append("|---|---|---|---|---|")
        for name, fmt in FORMATS:
            for gs in (128, 64, 32, 16):
                if isinstance(fmt, str):
                    codes, scales = amx.quantize_f16s(x, gs, fmt.endswith("-asym"), e4m3=fmt.startswith("e4m3"))
                    e = amx.quant_error_f16s(x, codes, scales, gs).cpu().numpy()
                else:
                    codes, scales = amx.quantize(x, gs, fmt)
                    e = amx.quant_error(x, codes, scales, gs).cpu().numpy()
                lines.append(f"| {name} | {gs} | {e[1] / e[0]:.3e} | {100 * e[2] / max(e[1], 1e-300):.1f} % | "
                             f"{100 * e[3] / x.numel():.2f} % |")
    return "\n".join(lines)


def kernel_rate(rows: int = 16384, K: int = 8192, iters: int = 20):
    """GB/s of amx_quant_error on a tensor larger than the L2 (bytes read: source, codes and scales)."""
    x = (torch.randn(rows, K, device="cuda") * 0.5).to(torch.bfloat16)
    codes, scales = amx.quantize(x, 32)
    L = amx.lib()
    out = torch.empty(4, dtype=torch.float64, device="cuda")
    ws = torch.empty(L.amx_quant_error_workspace_bytes(), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream

    def run():
        rc = L.amx_quant_error(x.data_ptr(), rows, K, K, codes.data_ptr(), scales.data_ptr(), 32, out.data_ptr(),
                               ws.data_ptr(), ws.numel(), stream)
        if rc:
            raise RuntimeError(amx.status_string(rc))

    for _ in range(3):
        run()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0.record()
    for _ in range(iters):
        run()
    t1.record()
    torch.cuda.synchronize()
    ms = t0.elapsed_time(t1) / iters
    return rows * K * 2.5625 / (ms * 1e-3) / 1e9, ms


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--rows", type=int, default=2048)
    args = ap.parse_args()
    build.build()
    print(report(args.rows))
    gbs, ms = kernel_rate()
    print(f"\namx_quant_error on 16384 x 8192: {ms * 1e3:.0f} us, {gbs:.0f} GB/s of source, codes and scales")
