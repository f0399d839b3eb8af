#!/usr/bin/env python
"""Benchmark of the AMXFP4 quantize + GEMM hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one pass over the 70B-shaped long-context prefill linears (M = 16384 tokens; 8192->10240,
8192->28672, 28672->8192 - the largest of the linear-layer workloads that fits one GPU): for every layer
the bf16 activation and the bf16 weight are cast to AMXFP4 and multiplied with fp32 accumulation.
Inputs are seeded synthetic tensors (channel outliers) resident in HBM.  Prints one JSON line.
--config 2 / 3 time the smaller linear workloads the same way.

With N > 1 (launched by torch.distributed.run) every rank runs the same token batch shape on its
own GPU (token-row sharding of a larger batch: no data-path collective), and the value is the
aggregate over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

CONFIG = 4          # the largest single-GPU linear workload; --config 2 / 3 time the smaller ones
WORKLOADS = {2: "config 2: LLaMA-7B-shaped prefill linears, M=2048, 4 layers",
             3: "config 3: LLaMA-3-8B-shaped prefill linears, M=8192, 4 layers (SiLU-skewed activations)",
             4: "config 4: 70B-scale prefill linears, M=16384, 3 layers"}
GS = 32
NOMINAL_FP4_TFLOPS = 9000.0      # NVIDIA's dense FP4 figure for one B200 (HGX B200 data sheet)
NOMINAL_HBM_GBS = 8000.0
BYTES_PER_ELEM = 2.0 + 0.5 + 2.0 / 32.0   # bf16 read + 4-bit code + two scale bytes per 32
# what the step's cast moves: bf16 read, two sign planes, two scale bytes and four scale-factor bytes per 32 (the
# canonical codes are not written: the step only multiplies)
MOVED_BYTES_PER_ELEM = 2.0 + 1.0 + 2.0 / 32.0 + 4.0 / 32.0
# DRAM bytes (read + write) per GEMM launch of the FP4 kernel, mean over the layers of a config, from the ncu
# captures summarised in profiles/ (None: no capture of the current kernel on that config).
GEMM_DRAM_TRAFFIC_PER_LAUNCH = {2: 89.2e6, 3: 613.7e6, 4: 4.225e9}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d["bf16_tflops_sustained"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def layer_shapes():
    from paper_2411_09909_b200 import inputs
    spec = inputs.LINEAR_CONFIGS[CONFIG]
    return spec["M"], spec["layers"]


def total_flops():
    M, layers = layer_shapes()
    return sum(2.0 * M * N * K for K, N in layers)


def quantized_elements():
    M, layers = layer_shapes()
    return sum(M * K + N * K for K, N in layers)


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=self.file, stderr=subprocess.DEVNULL)
        except OSError:
            pass

    def mark(self):
        """Samples written before this call (warm-up, idle) are ignored by stop()."""
        self.file.flush()
        self.skip = sum(1 for l in open(self.file.name) if l.strip())

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.file.flush()
        rows = [l.strip().split(", ") for l in open(self.file.name) if l.strip()][getattr(self, "skip", 0):]
        os.unlink(self.file.name)
        sm, reasons = [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 6:
                continue
            try:
                sm.append(float(r[0]))
                out["sm_max_mhz"] = float(r[1])
            except ValueError:
                continue
            for name, v in zip(names, r[2:6]):
                if v.strip().lower() == "active":
                    reasons.add(name)
        if sm:
            busy = [v for v in sm if v >= 0.5 * max(sm)]
            out["sm_mhz"] = float(np.median(busy))
        out["reasons"] = sorted(reasons)
        out["samples"] = len(sm)
        return out


def cpu_baseline(sample_rows: int = 2048, layer: int = 0):
    """The oracle, as it stands, on the host cores: quantize a row sample of the activation and the whole
    weight of one layer, then the fp64 product of that sample."""
    import oracle
    from paper_2411_09909_b200 import inputs
    K, N = inputs.LINEAR_CONFIGS[CONFIG]["layers"][layer]
    a = inputs.activation(CONFIG, layer, M=sample_rows)
    w = inputs.weight(CONFIG, layer)
    oracle.lib()
    t0 = time.perf_counter()
    qa = oracle.quantize(a, GS)
    qw = oracle.quantize(w, GS)
    t1 = time.perf_counter()
    oracle.gemm(*qa, *qw, GS)
    t2 = time.perf_counter()
    flops = 2.0 * sample_rows * N * K
    return {
        "value": flops / (t2 - t0) / 1e12, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
        "sample": f"config {CONFIG} layer {layer} ({K}->{N}): {sample_rows} token rows x all N x all K; "
                  f"quantize of the sample activation and the whole weight, then the fp64 product",
        "seconds": t2 - t0,
        "quantize_melem_per_s": (a.size + w.size) / (t1 - t0) / 1e6,
    }


def run_reference(args):
    """Reference arm: the CPU oracle on bounded samples of the same workload, rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    for _ in range(max(args.warmup, 0)):
        cpu_baseline(sample_rows=8)
    runs = [cpu_baseline(sample_rows=256) for _ in range(args.steps)]
    secs = float(np.mean([r["seconds"] for r in runs]))
    val = float(np.mean([r["value"] for r in runs]))
    base = dict(runs[-1], value=val)
    line = {
        "impl": "reference", "metric": "AMXFP4 quant+GEMM TFLOPS", "value": val, "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": secs * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOADS[CONFIG] + " (bounded sample per step: 256 token rows of layer 0)"},
        "cpu_baseline": base,
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def time_attention(heads: int, iters: int = 3):
    """Config 5 (heads x 8192 x 128, non-causal) through amx_attention: milliseconds per call."""
    import torch
    from paper_2411_09909_b200 import amx, inputs
    L = amx.lib()
    L5, D5 = 8192, 128
    q5, k5, v5 = (torch.from_numpy(t.view(np.int16)).cuda().view(torch.bfloat16) for t in inputs.attention_qkv(heads, L5))
    ws5 = torch.empty(L.amx_attention_workspace_bytes(L5, D5), dtype=torch.uint8, device="cuda")
    o5 = torch.empty((heads, L5, D5), dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream

    def attn(flags=0):
        rc = L.amx_attention(q5.data_ptr(), k5.data_ptr(), v5.data_ptr(), heads, L5, D5, flags, o5.data_ptr(),
                             ws5.data_ptr(), ws5.numel(), stream)
        if rc != 0:
            raise RuntimeError(amx.status_string(rc))

    def timed(flags):
        attn(flags)
        torch.cuda.synchronize()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for _ in range(iters):
            attn(flags)
        a1.record()
        torch.cuda.synchronize()
        return a0.elapsed_time(a1) / iters

    a_ms = timed(0)
    c_ms = timed(amx.ATTN_CAUSAL)
    return {"workload": f"config 5: {heads} heads x {L5} x {D5}, non-causal; Q, K, V and the attention map all cast to AMXFP4",
            "ms": a_ms, "useful_tflops": 4.0 * heads * L5 * L5 * D5 / (a_ms * 1e-3) / 1e12, "ms_per_head": a_ms / heads,
            "causal": {"ms": c_ms, "what": "the same call with AMX_ATTN_CAUSAL (not the benchmark's configuration): blocks of "
                                           "keys after their queries are skipped in all three products"}}


def time_decode(steps: int, A=None, W=None):
    """Decode-like shape: 16 token rows against the config-2 weights (cast once), amx_quant_gemm per layer, replayed as
    a CUDA graph.  Bound by streaming the 4.5-bit weights: reports the rate at which they are read."""
    import torch
    from paper_2411_09909_b200 import amx, inputs
    L = amx.lib()
    peaks = measured_peaks()
    layers = inputs.LINEAR_CONFIGS[2]["layers"]
    if A is None:
        def to_dev(bits):
            return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
        A = [to_dev(inputs.activation(2, li, M=64)) for li in range(len(layers))]
        W = [to_dev(inputs.weight(2, li)) for li in range(len(layers))]
    stream = torch.cuda.current_stream().cuda_stream

    def check(rc):
        if rc != 0:
            raise RuntimeError(amx.status_string(rc))

    REPS = 3                          # distinct copies of the weights: 3 x 88 MB of codes and scales exceed the L2

    def time_rows(Md):
        dd = []
        for li, (K, N) in enumerate(layers):
            wc_, ws_ = amx.quantize(W[li], GS)
            ad = A[li][:Md].contiguous()
            need = max(L.amx_quant_gemm_workspace_bytes(Md, N, K, GS, 0), 256)
            dd.append((ad, [(wc_.clone(), ws_.clone()) for _ in range(REPS)],
                       torch.empty((Md, N), dtype=torch.float32, device="cuda"),
                       torch.empty(need, dtype=torch.uint8, device="cuda")))
            del wc_, ws_

        def decode_step(stream, rep=0):
            for li, (K, N) in enumerate(layers):
                ad, wq, cd, wsd = dd[li]
                wc_, ws_ = wq[rep]
                check(L.amx_quant_gemm(ad.data_ptr(), K, wc_.data_ptr(), ws_.data_ptr(), None, 0, Md, N, K, GS, 0,
                                       cd.data_ptr(), N, wsd.data_ptr(), wsd.numel(), stream))

        decode_step(stream)
        torch.cuda.synchronize()
        sd = torch.cuda.Stream()
        sd.wait_stream(torch.cuda.current_stream())
        gd = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gd, stream=sd):
            for rep in range(REPS):
                decode_step(torch.cuda.current_stream().cuda_stream, rep)
        for _ in range(3):
            gd.replay()
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        d0.record()
        for _ in range(steps):
            gd.replay()
        d1.record()
        torch.cuda.synchronize()
        return d0.elapsed_time(d1) / (steps * REPS) * 1e3, dd

    Md = 16
    d_us, dd = time_rows(Md)
    decode_kernel = L.amx_gemm_kernel_for(Md, layers[0][1], layers[0][0], GS, 0)
    more_rows = {}
    for rows_ in (32, 64):
        if all(a.shape[0] >= rows_ for a in A):
            more_rows[str(rows_)] = time_rows(rows_)[0]
    w_bytes = sum(N * K for K, N in layers) * (0.5 + 2.0 / 32.0)
    # the same with the weights prepared once for the FP4 kernel (amx_quantize_prepared + amx_gemm_prepared)
    dp = []
    cw_ = [torch.empty((N, K // 2), dtype=torch.uint8, device="cuda") for K, N in layers]
    cs_ = [torch.empty((N, K // GS, 2), dtype=torch.uint8, device="cuda") for K, N in layers]
    for li, (K, N) in enumerate(layers):
        pw_ = torch.empty(L.amx_prepared_bytes(N, K, GS, 1), dtype=torch.uint8, device="cuda")
        check(L.amx_quantize_prepared(W[li].data_ptr(), N, K, GS, 1, cw_[li].data_ptr(), cs_[li].data_ptr(),
                                      pw_.data_ptr(), pw_.numel(), stream))
        dp.append((pw_, torch.empty(L.amx_prepared_bytes(Md, K, GS, 0), dtype=torch.uint8, device="cuda"),
                   torch.empty((Md, K // 2), dtype=torch.uint8, device="cuda"),
                   torch.empty((Md, K // GS, 2), dtype=torch.uint8, device="cuda"),
                   torch.empty(max(L.amx_gemm_prepared_workspace_bytes(Md, N, K, GS), 256), dtype=torch.uint8, device="cuda")))

    def decode_prepared_step(stream):
        for li, (K, N) in enumerate(layers):
            ad, _, cd, _ = dd[li]
            pw_, pa_, ac_, as_, wsp = dp[li]
            check(L.amx_quantize_prepared(ad.data_ptr(), Md, K, GS, 0, ac_.data_ptr(), as_.data_ptr(), pa_.data_ptr(),
                                          pa_.numel(), stream))
            check(L.amx_gemm_prepared(pa_.data_ptr(), pw_.data_ptr(), Md, N, K, GS, cd.data_ptr(), N, wsp.data_ptr(),
                                      wsp.numel(), stream))

    decode_prepared_step(stream)
    torch.cuda.synchronize()
    sp = torch.cuda.Stream()
    sp.wait_stream(torch.cuda.current_stream())
    gp = torch.cuda.CUDAGraph()
    with torch.cuda.graph(gp, stream=sp):
        decode_prepared_step(torch.cuda.current_stream().cuda_stream)
    for _ in range(3):
        gp.replay()
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    p0.record()
    for _ in range(steps):
        gp.replay()
    p1.record()
    torch.cuda.synchronize()
    dp_us = p0.elapsed_time(p1) / steps * 1e3
    del dp
    decode = {"workload": f"{Md} token rows x the four config-2 weights (cast once; {REPS} copies of the weights in turn, "
                          "so that they come from HBM, not from the L2); amx_quant_gemm per layer, graph replay",
              "prepared_weights": {"us_per_step": dp_us,
                                   "what": "weights prepared once for the FP4 kernel (1.06 B/element resident), per layer "
                                           "amx_quantize_prepared of the rows + amx_gemm_prepared with K ranges",
                                   "weight_gb_per_s_canonical_bytes": sum(N * K for K, N in layers) * 0.5625 / (dp_us * 1e-6) / 1e9},
              "us_per_step": d_us, "weight_gb_per_s": w_bytes / (d_us * 1e-6) / 1e9,
              "frac_of_measured_copy": w_bytes / (d_us * 1e-6) / 1e9 / peaks["hbm_gbs"],
              "launches_per_step": 2 * len(layers),
              "us_per_step_more_rows": more_rows,
              "kernel": ("weight-streaming kernel (canonical weights read once, exact bf16 decode, mma.sync; K ranges "
                         "added over a thread-block cluster)" if decode_kernel == amx.GEMM_ROWS
                         else "tcgen05 kind::f16 (bf16 decode), K cut into slices over CTAs")}
    return decode


def run_ours(args):
    import torch
    from paper_2411_09909_b200 import amx, inputs, build, sharding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    build.build()
    L = amx.lib()
    peaks = measured_peaks()
    M, layers = layer_shapes()
    gemm_flag = {"auto": 0, "simt": 0x10, "tc": 0x20, "fp4": 0x40}[args.gemm]
    keep = [int(t) for t in args.layers.split(",") if t != ""] or list(range(len(layers)))
    layer_ids = keep
    layers = [layers[i] for i in keep]
    flops_step = sum(2.0 * M * N * K for K, N in layers)
    elems_step = sum(M * K + N * K for K, N in layers)
    use_graph = args.graph or (CONFIG == 2 and not args.no_graph)

    def to_dev(bits):
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)

    # ---- resident inputs and preallocated outputs
    A, W, bufs = [], [], []
    host = []
    for li, (K, N) in enumerate(layers):
        a_bits, w_bits = inputs.activation(CONFIG, layer_ids[li]), inputs.weight(CONFIG, layer_ids[li])
        host.append((a_bits, w_bits))
        A.append(to_dev(a_bits))
        W.append(to_dev(w_bits))
        ws_bytes = max(L.amx_workspace_bytes(M, N, K, GS, gemm_flag), 256)
        bufs.append({
            "ac": torch.empty((M, K // 2), dtype=torch.uint8, device="cuda"),
            "as": torch.empty((M, K // GS, 2), dtype=torch.uint8, device="cuda"),
            "wc": torch.empty((N, K // 2), dtype=torch.uint8, device="cuda"),
            "ws": torch.empty((N, K // GS, 2), dtype=torch.uint8, device="cuda"),
            "c": torch.empty((M, N), dtype=torch.float32, device="cuda"),
            "work": torch.empty(ws_bytes, dtype=torch.uint8, device="cuda"),
        })
    stream = torch.cuda.current_stream().cuda_stream
    fused_prepare = L.amx_gemm_kernel_for(M, layers[0][1], layers[0][0], GS, gemm_flag) == 0x40 and not args.unfused
    if fused_prepare:
        for li, (K, N) in enumerate(layers):
            bufs[li]["pa"] = torch.empty(L.amx_prepared_bytes(M, K, GS, 0), dtype=torch.uint8, device="cuda")
            bufs[li]["pw"] = torch.empty(L.amx_prepared_bytes(N, K, GS, 1), dtype=torch.uint8, device="cuda")
    gemm_kernel = {0x10: "simt", 0x20: "tcgen05 kind::f16 (bf16 decode)", 0x40: "tcgen05 kind::mxf4nvf4 (sign split)"}[
        L.amx_gemm_kernel_for(M, layers[0][1], layers[0][0], GS, gemm_flag)]

    def check(rc):
        if rc != 0:
            raise RuntimeError(amx.status_string(rc))

    # --format: the step in one of the symmetric comparison formats (profiling aid; the bench line is AMXFP4)
    step_fmt = {"amxfp4": amx.FMT_AMXFP4, "sym_fp8": amx.FMT_SYM_FP8, "mxfp4": amx.FMT_MXFP4}[args.format]

    def cast_a(li, st):
        K, N = layers[li]
        b = bufs[li]
        if fused_prepare:   # the cast writes the FP4 kernel's operand (sign planes, scale factors) in the same pass
            check(L.amx_quantize_prepared_fmt(A[li].data_ptr(), M, K, GS, 0, step_fmt, None, b["as"].data_ptr(),
                                              b["pa"].data_ptr(), b["pa"].numel(), st))
        else:
            check(L.amx_quantize_fmt(A[li].data_ptr(), M, K, K, GS, step_fmt, b["ac"].data_ptr(), b["as"].data_ptr(), st))

    def cast_w(li, st):
        K, N = layers[li]
        b = bufs[li]
        if fused_prepare:
            check(L.amx_quantize_prepared_fmt(W[li].data_ptr(), N, K, GS, 1, step_fmt, None, b["ws"].data_ptr(),
                                              b["pw"].data_ptr(), b["pw"].numel(), st))
        else:
            check(L.amx_quantize_fmt(W[li].data_ptr(), N, K, K, GS, step_fmt, b["wc"].data_ptr(), b["ws"].data_ptr(), st))

    def gemm(li, st, sym=step_fmt != amx.FMT_AMXFP4):
        K, N = layers[li]
        b = bufs[li]
        if fused_prepare:      # sym: both operands are single planes, the one-plane pipeline of the same kernel
            fn = L.amx_gemm_prepared_sym if sym else L.amx_gemm_prepared
            check(fn(b["pa"].data_ptr(), b["pw"].data_ptr(), M, N, K, GS, b["c"].data_ptr(), N,
                     b["work"].data_ptr(), b["work"].numel(), st))
        else:
            check(L.amx_gemm(b["ac"].data_ptr(), b["as"].data_ptr(), b["wc"].data_ptr(), b["ws"].data_ptr(),
                             M, N, K, GS, gemm_flag, b["c"].data_ptr(), N, b["work"].data_ptr(), b["work"].numel(), st))

    # Schedules of one step.  Every one records, when asked, CUDA events around the cast phase and the GEMM of each
    # layer on the main stream (the stream the GEMM is launched on): the roofline of the GEMM kernel is taken from
    # those events inside the timed region.
    #   serial   one stream, kernels in order
    #   pair     within a layer the cast of the activation and the cast of the weight run side by side (two
    #            streams): they are independent inputs of the same GEMM in any model, and the small activation cast
    #            fills the tail of the weight cast's last wave.  Layers stay in order.
    #   overlap  all weight casts on a second stream, running ahead of the GEMMs of earlier layers (they depend on
    #            nothing the step computes); not the default: in a model only the weights are available ahead
    cast_stream = torch.cuda.Stream() if args.schedule in ("pair", "overlap") else None

    def run_step(events=None):
        main = torch.cuda.current_stream()
        ms = main.cuda_stream
        ready = []
        if args.schedule == "overlap":
            cast_stream.wait_stream(main)
            for li in range(len(layers)):
                cast_w(li, cast_stream.cuda_stream)
                ev = torch.cuda.Event()
                ev.record(cast_stream)
                ready.append(ev)
        for li in range(len(layers)):
            if events is not None:
                e0, e1, e2 = events[li]
                e0.record(main)
            if args.schedule == "pair":
                cast_stream.wait_stream(main)
                cast_a(li, cast_stream.cuda_stream)
                cast_w(li, ms)
                main.wait_stream(cast_stream)
            elif args.schedule == "overlap":
                cast_a(li, ms)
                main.wait_event(ready[li])
            else:
                cast_a(li, ms)
                cast_w(li, ms)
            if events is not None:
                e1.record(main)
            gemm(li, ms)
            if events is not None:
                e2.record(main)
        if args.schedule == "overlap":
            main.wait_stream(cast_stream)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    def new_events():
        return [tuple(torch.cuda.Event(enable_timing=True) for _ in range(3)) for _ in layers]

    sampler = ClockSampler(local) if rank == 0 else None   # started early: nvidia-smi needs ~0.2 s to begin
    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        run_step()
    barrier()
    if sampler:
        time.sleep(0.3)
        sampler.mark()
    # Plain launches with events between the kernels by default; --graph (the default for the small config 2, whose
    # step is launch-bound in places) replays a CUDA graph of one step, and the per-kernel times then come from a
    # separate pass of plain launches.
    graph = None
    if use_graph:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            run_step()
        for _ in range(3):
            graph.replay()
        barrier()
    step_events = [new_events() for _ in range(args.steps)] if graph is None else []
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_start.record()
    for i in range(args.steps):
        if graph is not None:
            graph.replay()
        else:
            run_step(step_events[i])
    t_end.record()
    barrier()
    elapsed_ms = t_start.elapsed_time(t_end)
    clocks = sampler.stop() if sampler else None
    elapsed_ms = sharding.max_over_ranks(elapsed_ms, "cuda")      # the slowest rank's time
    # a kernel that gave up on a bounded wait must not be reported as a fast run
    for li in range(len(layers)):
        st_word = amx.gemm_status(bufs[li]["work"])
        if st_word != 0:
            raise RuntimeError(f"layer {layer_ids[li]}: GEMM status {amx.status_string(st_word)}")
    if graph is not None:
        event_steps = min(args.steps, 50)
        step_events = [new_events() for _ in range(event_steps)]
        for ev in step_events:
            run_step(ev)
        torch.cuda.synchronize()
    # per layer: mean duration of the cast phase and of the GEMM launch over the timed steps
    q_ms_layer = [float(np.mean([ev[li][0].elapsed_time(ev[li][1]) for ev in step_events])) for li in range(len(layers))]
    g_ms_layer = [float(np.mean([ev[li][1].elapsed_time(ev[li][2]) for ev in step_events])) for li in range(len(layers))]
    q_ms, g_ms = sum(q_ms_layer), sum(g_ms_layer)     # per step

    def timed_graph(fn, steps):
        """Mean milliseconds of fn(stream) over `steps` replays of a CUDA graph of one call."""
        fn(stream)
        torch.cuda.synchronize()
        sg = torch.cuda.Stream()
        sg.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=sg):
            fn(torch.cuda.current_stream().cuda_stream)
        for _ in range(3):
            g.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps

    extra_steps = max(3, min(args.steps, 30 if CONFIG == 2 else 10))

    # ---- the inference-time variant: weights cast and prepared once, activations per step (reported beside
    # the headline, which casts both operands every step)
    weights_cached = None
    if fused_prepare and not args.layers:
        def cached_step(st):
            for li in range(len(layers)):
                cast_a(li, st)
                gemm(li, st)
        c_ms = sharding.max_over_ranks(timed_graph(cached_step, extra_steps), "cuda")
        weights_cached = {"value": sharding.aggregate_rate(flops_step, world, c_ms) / 1e12, "unit": "TFLOP/s",
                          "ms_per_step": c_ms,
                          "what": "weights cast and prepared once; per step: cast + prepare activations, GEMM"}

    # ---- the paper's symmetric comparison formats on the same kernels (one shared scale per group: no split by
    # sign, one FP4 product per tile pair instead of four).  Shows what AMXFP4's asymmetry costs on this GPU, and
    # the rate of the FP4 pipe on this kernel design when nothing is split.
    format_variants = None
    if fused_prepare and not args.layers and not args.skip_extras:
        format_variants = {}
        for name, fmt in (("sym_fp8", 1), ("mxfp4", 2)):
            def fmt_step(st, with_casts=True, fmt=fmt, sym=True):
                for li, (K, N) in enumerate(layers):
                    b = bufs[li]
                    if with_casts:
                        check(L.amx_quantize_prepared_fmt(A[li].data_ptr(), M, K, GS, 0, fmt, None,
                                                          b["as"].data_ptr(), b["pa"].data_ptr(), b["pa"].numel(), st))
                        check(L.amx_quantize_prepared_fmt(W[li].data_ptr(), N, K, GS, 1, fmt, None,
                                                          b["ws"].data_ptr(), b["pw"].data_ptr(), b["pw"].numel(), st))
                    gemm(li, st, sym)
            res = {}
            for key, with_casts, sym in (("step", True, True), ("gemm", False, True), ("gemm_general_kernel", False, False)):
                fmt_step(stream)
                v_ms = timed_graph(lambda st: fmt_step(st, with_casts, sym=sym), extra_steps)
                res[key + "_tflops"] = flops_step / (v_ms * 1e-3) / 1e12
                res[key + "_ms"] = v_ms
            format_variants[name] = res
            for li in range(len(layers)):                        # the one-plane promise held, no wait expired
                if amx.gemm_status(bufs[li]["work"]) != 0:
                    raise RuntimeError(f"{name}, layer {layer_ids[li]}: GEMM status {amx.status_string(amx.gemm_status(bufs[li]['work']))}")
        # the AMXFP4 GEMMs with a bf16 result (rounded in the epilogue: half the bytes stored); operands as the
        # headline step's casts left them
        run_step()
        def amx_gemms(st, out_flags=0):
            for li, (K, N) in enumerate(layers):
                b = bufs[li]
                check(L.amx_gemm_prepared_ex(b["pa"].data_ptr(), b["pw"].data_ptr(), M, N, K, GS, out_flags,
                                             b["c"].data_ptr(), N, b["work"].data_ptr(), b["work"].numel(), st))
        for name, out_flags in (("amxfp4_f32_result", 0), ("amxfp4_bf16_result", amx.PREP_OUT_BF16)):
            amx_gemms(stream, out_flags)
            v_ms = timed_graph(lambda st: amx_gemms(st, out_flags), extra_steps)
            format_variants[name] = {"gemm_tflops": flops_step / (v_ms * 1e-3) / 1e12, "gemm_ms": v_ms}
        # NVFP4 / ANVFP4 (group 16, E4M3 group scales + fp32 tensor scale: Section 5's comparison format): the scale
        # bytes are the tensor cores' native type, NVFP4 is one product per tile pair, ANVFP4 four
        nv = []
        for li, (K, N) in enumerate(layers):
            nv.append((torch.empty(L.amx_nvfp4_prepared_bytes(M, K, 0), dtype=torch.uint8, device="cuda"),
                       torch.empty(L.amx_nvfp4_prepared_bytes(N, K, 1), dtype=torch.uint8, device="cuda"),
                       torch.empty(2, dtype=torch.float32, device="cuda"), torch.empty(2, dtype=torch.float32, device="cuda")))
        for name, flag in (("nvfp4", 0), ("anvfp4", 1)):
            def nv_step(st, with_casts=True, flag=flag):
                for li, (K, N) in enumerate(layers):
                    pa, pw, ta, tw = nv[li]
                    b = bufs[li]
                    if with_casts:
                        check(L.amx_quantize_nvfp4(A[li].data_ptr(), M, K, K, flag, None, None, ta.data_ptr(), 0, pa.data_ptr(),
                                                   pa.numel(), st))
                        check(L.amx_quantize_nvfp4(W[li].data_ptr(), N, K, K, flag, None, None, tw.data_ptr(), 1, pw.data_ptr(),
                                                   pw.numel(), st))
                    check((L.amx_gemm_nvfp4 if flag else L.amx_gemm_nvfp4_sym)(
                        pa.data_ptr(), pw.data_ptr(), M, N, K, b["c"].data_ptr(), N, b["work"].data_ptr(), b["work"].numel(), st))
            res = {}
            for key, with_casts in (("step", True), ("gemm", False)):
                nv_step(stream)
                v_ms = timed_graph(lambda st: nv_step(st, with_casts), extra_steps)
                res[key + "_tflops"] = flops_step / (v_ms * 1e-3) / 1e12
                res[key + "_ms"] = v_ms
            format_variants[name] = res
            for li in range(len(layers)):                        # the one-plane promise held, no wait expired
                if amx.gemm_status(bufs[li]["work"]) != 0:
                    raise RuntimeError(f"{name}, layer {layer_ids[li]}: GEMM status {amx.status_string(amx.gemm_status(bufs[li]['work']))}")
        del nv
        format_variants["what"] = ("same workload and GEMM kernel with other formats: sym_fp8 / mxfp4 = the paper's symmetric "
                                   "comparison formats (amx_quantize_prepared_fmt), nvfp4 / anvfp4 = group 16 with E4M3 scales "
                                   "and a tensor scale (amx_quantize_nvfp4: two launches, the tensor maximum first); step = "
                                   "casts of both operands + GEMMs, gemm = the GEMMs alone; the symmetric formats run the "
                                   "one-plane pipeline (amx_gemm_prepared_sym, amx_gemm_nvfp4_sym), gemm_general_kernel = "
                                   "the same operands through amx_gemm_prepared; amxfp4_bf16_result = the headline's "
                                   "AMXFP4 GEMMs through amx_gemm_prepared_ex with AMX_PREP_OUT_BF16, amxfp4_f32_result = the same measurement "
                                   "(GEMMs alone, graph replay) with the fp32 result")
        run_step()                      # leave the buffers as the headline step writes them
        torch.cuda.synchronize()

    # ---- the cast alone on a tensor larger than L2 (config-4 activation shape, 16384 x 8192 = 268 MB of bf16)
    quant_large = None
    if not args.layers:
        qr, qk = 16384, 8192
        xq = to_dev(inputs.activation(4, 0, M=256)).repeat(qr // 256, 1).contiguous()
        qc = torch.empty((qr, qk // 2), dtype=torch.uint8, device="cuda")
        qs = torch.empty((qr, qk // GS, 2), dtype=torch.uint8, device="cuda")
        for _ in range(3):
            check(L.amx_quantize(xq.data_ptr(), qr, qk, qk, GS, qc.data_ptr(), qs.data_ptr(), stream))
        q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        q_iters = 20
        torch.cuda.synchronize()
        q0.record()
        for _ in range(q_iters):
            check(L.amx_quantize(xq.data_ptr(), qr, qk, qk, GS, qc.data_ptr(), qs.data_ptr(), stream))
        q1.record()
        torch.cuda.synchronize()
        q_us = q0.elapsed_time(q1) * 1e3 / q_iters
        gbs = qr * qk * BYTES_PER_ELEM / (q_us * 1e-6) / 1e9
        quant_large = {"shape": [qr, qk], "us": q_us, "gb_per_s": gbs,
                       "pct_of_nominal_hbm_8TBs": 100.0 * gbs / NOMINAL_HBM_GBS,
                       "frac_of_measured_copy": gbs / peaks["hbm_gbs"]}
        # the same tensor through the cast that writes the GEMM-ready operand (alone on the GPU, not beside a second cast)
        qp = torch.empty(L.amx_prepared_bytes(qr, qk, GS, 0), dtype=torch.uint8, device="cuda")

        def cast_prepared():
            check(L.amx_quantize_prepared(xq.data_ptr(), qr, qk, GS, 0, None, qs.data_ptr(), qp.data_ptr(), qp.numel(), stream))
        for _ in range(3):
            cast_prepared()
        torch.cuda.synchronize()
        q0.record()
        for _ in range(q_iters):
            cast_prepared()
        q1.record()
        torch.cuda.synchronize()
        qp_us = q0.elapsed_time(q1) * 1e3 / q_iters
        qp_gbs = qr * qk * MOVED_BYTES_PER_ELEM / (qp_us * 1e-6) / 1e9
        quant_large["prepared"] = {"us": qp_us, "gb_per_s_moved": qp_gbs, "frac_of_measured_copy": qp_gbs / peaks["hbm_gbs"]}
        del xq, qc, qs, qp

    # ---- config 5: fully quantized attention for all heads (32 x 8192 x 128), one call of amx_attention
    attention = None
    if not args.layers and not args.skip_extras and world == 1:
        attention = time_attention(32)

    # ---- config 1: one small layer (128 x 1024 -> 1024), latency-bound: microseconds per call of amx_quant_gemm,
    # with the weight cast ahead of time and with both operands cast in the call
    small_case = None
    if not args.layers and not args.skip_extras and world == 1:
        a1b, w1b = to_dev(inputs.activation(1, 0)), to_dev(inputs.weight(1, 0))
        w1c, w1s = amx.quantize(w1b, GS)
        M1, K1 = a1b.shape
        N1 = w1c.shape[0]
        c1 = torch.empty((M1, N1), dtype=torch.float32, device="cuda")
        ws1 = torch.empty(max(L.amx_quant_gemm_workspace_bytes(M1, N1, K1, GS, amx.WEIGHT_BF16), 256), dtype=torch.uint8,
                          device="cuda")

        def small(both):
            check(L.amx_quant_gemm(a1b.data_ptr(), K1, None if both else w1c.data_ptr(), None if both else w1s.data_ptr(),
                                   w1b.data_ptr() if both else None, K1 if both else 0, M1, N1, K1, GS, 0, c1.data_ptr(), N1,
                                   ws1.data_ptr(), ws1.numel(), stream))

        us = {}
        for both in (False, True):
            for _ in range(5):
                small(both)
            s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            s0.record()
            for _ in range(200):
                small(both)
            s1.record()
            torch.cuda.synchronize()
            us[both] = s0.elapsed_time(s1) * 1e3 / 200
        small_case = {"workload": f"config 1: A {M1}x{K1}, W {N1}x{K1}; one call of amx_quant_gemm",
                      "us_per_call": us[False], "us_per_call_both_operands_cast": us[True],
                      "note": "us_per_call: the weight was cast ahead of time; both_operands_cast: the bf16 weight is "
                              "cast in the same call.  Launch-latency-bound (32 output tiles at most): microseconds, "
                              "not a roofline fraction"}

    # ---- decode-like shape: 16 token rows against the config-2 weights (see time_decode)
    decode = None
    if not args.layers and not args.skip_extras and world == 1:
        decode = time_decode(max(20, min(args.steps, 100)))

    # ---- end to end through the host-buffer entry point (pinned host tensors, copies inside the timing).
    # amx_linear_host_pipelined per layer on three streams (copies in, kernels, copies out), a workspace per layer,
    # no synchronisation between the layers (AMX_HOST_NO_SYNC): the rows of A go through in chunks, so results go
    # back to the host while later rows and the next layer's inputs come in.
    e2e = None
    if (rank == 0 or world > 1) and not args.skip_extras:
        pinned = []
        for li, (K, N) in enumerate(layers):
            a_bits, w_bits = host[li]
            pinned.append((torch.from_numpy(a_bits.view(np.int16)).view(torch.bfloat16).pin_memory(),
                           torch.from_numpy(w_bits.view(np.int16)).view(torch.bfloat16).pin_memory(),
                           torch.empty((M, N), dtype=torch.float32).pin_memory()))
        lh_ws = [torch.empty(L.amx_linear_host_pipelined_workspace_bytes(M, N, K, GS, gemm_flag), dtype=torch.uint8, device="cuda")
                 for K, N in layers]
        lh_streams = [torch.cuda.Stream() for _ in range(3)]

        def e2e_step():
            for li, (K, N) in enumerate(layers):
                a, w, c = pinned[li]
                check(L.amx_linear_host_pipelined(a.data_ptr(), w.data_ptr(), M, N, K, GS, gemm_flag | amx.HOST_NO_SYNC,
                                                  c.data_ptr(), lh_ws[li].data_ptr(), lh_ws[li].numel(),
                                                  *(s.cuda_stream for s in lh_streams)))
            torch.cuda.synchronize()

        e2e_step()
        for li in range(len(layers)):
            st_word = L.amx_linear_host_pipelined_status(lh_ws[li].data_ptr(), lh_streams[1].cuda_stream)
            if st_word != 0:
                raise RuntimeError(f"end-to-end leg, layer {layer_ids[li]}: status {amx.status_string(st_word)}")
        barrier()
        e2e_steps = max(2, min(args.steps, 5))
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_step()
        e2e_s = (time.perf_counter() - t0) / e2e_steps
        e2e_s = sharding.max_over_ranks(e2e_s, "cuda")
        e2e = {"value": world * flops_step / e2e_s / 1e12, "unit": "TFLOP/s",
               "h2d_bytes_per_step": int(elems_step * 2),
               "d2h_bytes_per_step": int(sum(M * N * 4 for _, N in layers)),
               "ms_per_step": e2e_s * 1e3,
               "what": "amx_linear_host_pipelined per layer from pinned host buffers on three streams (copies in, "
                       "kernels, copies out): the rows of A go through in chunks of 2048, so host-to-device and "
                       "device-to-host copies overlap within and across layers; PCIe-bound"}
        del pinned, lh_ws

    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return

    ms_per_step = elapsed_ms / args.steps
    value = sharding.aggregate_rate(flops_step, world, ms_per_step) / 1e12
    gemm_tflops = flops_step / (g_ms * 1e-3) / 1e12
    quant_gbs = elems_step * BYTES_PER_ELEM / (q_ms * 1e-3) / 1e9
    moved = MOVED_BYTES_PER_ELEM if fused_prepare else BYTES_PER_ELEM
    # Roofline denominator of the GEMM: 4 x the measured bf16 cuBLAS rate (nominal FP4 : bf16 ratio).  Which bf16
    # figure applies depends on the run: a timed region that stayed at (nearly) full clock without the power cap is
    # a burst, anything else is sustained.  Both fractions are printed.
    sm, sm_max = (clocks or {}).get("sm_mhz"), (clocks or {}).get("sm_max_mhz")
    burst = bool(sm and sm_max and sm >= 0.95 * sm_max and "sw_power_cap" not in (clocks or {}).get("reasons", []))
    peak_burst, peak_sust = 4.0 * peaks["bf16_tflops"], 4.0 * peaks["bf16_tflops_sustained"]
    fp4_peak = peak_burst if burst else peak_sust
    line = {
        "metric": "AMXFP4 quant+GEMM TFLOPS", "value": value, "unit": "TFLOP/s", "n_gpus": world,
        "steps": args.steps, "warmup": warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "fp4xfp4->f32",
        "data": "synthetic",
        "config": {"workload": (WORKLOADS[CONFIG] + "; activations and weights both cast to AMXFP4 every step, then GEMM"
                                + ("" if args.format == "amxfp4" else f" [comparison format {args.format} instead of AMXFP4]")),
                   "group_size": GS, "gemm_kernel": gemm_kernel,
                   "entry_points": "amx_quantize_prepared + amx_gemm_prepared" if fused_prepare else "amx_quantize + amx_gemm",
                   "l2": f"per-step inputs (~{int(elems_step * 2 / 1e6)} MB of bf16) exceed the 126 MB L2",
                   "launch": "CUDA graph of one step, replayed" if use_graph else "plain launches, CUDA events between the kernels",
                   "schedule": {"overlap": "weight casts on a second stream, overlapping the GEMMs of earlier layers",
                                "pair": "layers in order; a layer's two casts side by side on two streams",
                                "serial": "one stream, kernels in order"}[args.schedule]},
        "pct_of_nominal_fp4_peak": 100.0 * value / world / NOMINAL_FP4_TFLOPS,
        "nominal_fp4_peak_tflops": NOMINAL_FP4_TFLOPS,
        "gemm": {"useful_tflops": gemm_tflops, "ms_per_step": g_ms, "ms_per_layer": g_ms_layer,
                 # the sign split issues four FP4 products per useful one
                 "issued_tflops": gemm_tflops * (4.0 if "mxf4" in gemm_kernel else 1.0),
                 "pct_of_nominal_fp4_peak": 100.0 * gemm_tflops / NOMINAL_FP4_TFLOPS},
        "roofline": {"bound": "tensor", "achieved": gemm_tflops, "peak": fp4_peak, "unit": "TFLOP/s",
                     "frac": gemm_tflops / fp4_peak, "traffic": GEMM_DRAM_TRAFFIC_PER_LAUNCH.get(CONFIG),
                     "frac_burst": gemm_tflops / peak_burst, "frac_sustained": gemm_tflops / peak_sust,
                     "regime": "burst" if burst else "sustained",
                     "exact_mapping_ceiling_frac": 0.25,
                     "kernel": f"amx_gemm ({gemm_kernel})",
                     "timing": ("CUDA events around every GEMM launch inside the timed region" if not use_graph else
                                "CUDA events around every GEMM launch in a pass of plain launches after the timed graph replays"),
                     "peak_source": f"4 x {'burst' if burst else 'sustained'} bf16 cuBLAS rate ({peaks['source']}), nominal "
                                    "FP4:bf16 ratio; burst when the sampled SM clock stayed within 5 % of its maximum with "
                                    "no power cap",
                     # the HBM-bound kernel of the step: the cast
                     "quantize": {"bound": "hbm", "unit": "GB/s", "peak": peaks["hbm_gbs"],
                                  "peak_source": f"copy rate ({peaks['source']})",
                                  "prepared_cast": {"bytes_per_element": moved, "achieved": quant_gbs * moved / BYTES_PER_ELEM,
                                                    "frac": quant_gbs * moved / BYTES_PER_ELEM / peaks["hbm_gbs"],
                                                    "achieved_canonical_bytes": quant_gbs,
                                                    "what": "both casts of every layer of the step (events around the cast "
                                                            "phase); bytes actually moved per element: 2 read, 1 of sign "
                                                            "planes, 0.0625 of scale bytes, 0.125 of scale factors (the "
                                                            "canonical codes are not written)"},
                                  "prepared_cast_alone": (None if quant_large is None else
                                                          {"bytes_per_element": moved,
                                                           "achieved": quant_large["prepared"]["gb_per_s_moved"],
                                                           "frac": quant_large["prepared"]["frac_of_measured_copy"],
                                                           "what": "amx_quantize_prepared on 16384 x 8192 with nothing else "
                                                                   "running (in the step two casts share the GPU)"}),
                                  "plain_cast": (None if quant_large is None else
                                                 {"bytes_per_element": BYTES_PER_ELEM, "achieved": quant_large["gb_per_s"],
                                                  "frac": quant_large["frac_of_measured_copy"],
                                                  "pct_of_nominal_hbm_8TBs": quant_large["pct_of_nominal_hbm_8TBs"],
                                                  "what": "amx_quantize on 16384 x 8192 (268 MB of bf16)"})}},
        "quantize": {"gb_per_s": quant_gbs, "pct_of_nominal_hbm_8TBs": 100.0 * quant_gbs / NOMINAL_HBM_GBS,
                     "frac_of_measured_copy": quant_gbs / peaks["hbm_gbs"], "bytes_per_element": BYTES_PER_ELEM,
                     "ms_per_step": q_ms, "ms_per_layer": q_ms_layer, "large_tensor": quant_large,
                     "bytes_per_element_moved": moved, "gb_per_s_moved": quant_gbs * moved / BYTES_PER_ELEM},
        "weights_cached": weights_cached,
        "format_variants": format_variants,
        "attention": attention,
        "small_case": small_case,
        "decode": decode,
        "clocks": clocks,
        "e2e": e2e,
        # kernels per layer: 2 casts + the GEMM; without the fused entry points the FP4 kernel's operands need
        # one preparation kernel each on top
        "gpu_launches": (5 if "mxf4" in gemm_kernel and not fused_prepare else 3) * len(layers) * args.steps,
    }
    if len(layer_ids) != len(inputs.LINEAR_CONFIGS[CONFIG]["layers"]):
        line["config"]["layers"] = layer_ids
    if world == 1 and not args.skip_extras:
        line["cpu_baseline"] = cpu_baseline()
    print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--gemm", default="auto", choices=["auto", "simt", "tc", "fp4"], help="GEMM kernel to time")
    ap.add_argument("--unfused", action="store_true", help="amx_quantize + amx_gemm instead of the fused-preparation entry points")
    ap.add_argument("--schedule", choices=["serial", "pair", "overlap"], default="pair",
                    help="pair (default): a layer's two casts side by side, layers in order; serial: one stream; "
                         "overlap: weight casts on a second stream, running ahead of the GEMMs")
    ap.add_argument("--graph", action="store_true", help="time replays of a CUDA graph of one step (the default for config 2)")
    ap.add_argument("--no-graph", action="store_true", help="config 2: time plain launches instead of the graph")
    ap.add_argument("--format", default="amxfp4", choices=["amxfp4", "sym_fp8", "mxfp4"],
                    help="cast format of the step (profiling aid: the symmetric comparison formats need one FP4 product per tile pair)")
    ap.add_argument("--layers", default="", help="comma-separated layer indices to run (profiling aid; default all)")
    ap.add_argument("--skip-extras", action="store_true", help="skip the e2e and cpu_baseline legs (profiling aid)")
    ap.add_argument("--attention-only", action="store_true", help="time only the config-5 attention call (profiling aid)")
    ap.add_argument("--heads", type=int, default=32, help="heads for --attention-only")
    ap.add_argument("--decode-only", action="store_true", help="time only the 16-row decode step (profiling aid)")
    ap.add_argument("--config", type=int, default=4, choices=[2, 3, 4],
                    help="linear-layer workload (default 4, the largest that fits one GPU; 2 and 3 are smaller)")
    args = ap.parse_args()
    global CONFIG
    CONFIG = args.config
    if args.attention_only:
        import torch
        from paper_2411_09909_b200 import build
        torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
        build.build()
        print(json.dumps({"attention": time_attention(args.heads, iters=1)}))
    elif args.decode_only:
        import torch
        from paper_2411_09909_b200 import build
        torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
        build.build()
        print(json.dumps({"decode": time_decode(args.steps)}))
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
