#!/usr/bin/env python
"""Benchmark of the pattern-sparse 3x3 convolution path on B200.

A step is one pass of the whole hot path over one batch: the 13 pattern-pruned 3x3 convolutions of a VGG-16-shaped
stack (2x2 max-pools between blocks), batch 32 per GPU, fp32, 8 patterns, connectivity pruning 0 % in layer 1 and
60 % in the others, seeded synthetic weights and inputs.  The metric is effective GFLOP/s counting only the
multiply-accumulates on kept weights (2 * 4 * K * H * W * N flop per layer).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--batch B] [--no-extras]

Under torchrun every rank runs the same stack on its own batch (weak scaling, no data-path collective); the time is
the maximum over ranks.  ``--impl reference`` times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

FP32_LANES = 128                      # FP32 FMA lanes per SM on this architecture
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel (conv_umma_halo_kernel on the
# 256 -> 256 @ 56x56 layer): 28.5 MB in the ncu capture at batch 8 (profiles/conv_umma_halo_kernel_vgg16_L06_n8.txt),
# scaled by the units of a batch-32 launch (x4; reads grow in proportion, the output additionally leaves L2 at that size)
TRAFFIC_BYTES_PER_LAUNCH = 104771072 + 52571392
TRAFFIC_NOTE = ("dominant kernel (conv_umma_halo_kernel, 256 -> 256 @ 56x56, the form it has inside the stack): "
                "dram__bytes_read + dram__bytes_write of one launch at the benchmark's batch 32, one ncu capture "
                "(profiles/conv_umma_halo_kernel_vgg16_L06_n32.txt); algorithmic bytes of that launch: 102.8 MB split input + "
                "2.4 MB weights + 102.8 MB output, of which ~50 MB were still in L2 when the kernel ended")


def alu_peak_tflops(torch=None):
    """FP32 CUDA-core peak the kept-weight roofline is quoted against: SMs x 128 FMA lanes x 2 flop x max SM clock."""
    sms, ghz = 148, 1.965
    peaks = measured_peaks()[0]
    if peaks.get("sm_max_mhz"):
        ghz = float(peaks["sm_max_mhz"]) / 1e3
    if torch is not None and torch.cuda.is_available():
        sms = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
    return sms * FP32_LANES * 2 * ghz / 1e3


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            return json.load(fh), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], None, set()
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
            except (ValueError, IndexError):
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        busy = [c for c in sm if mx and c > 0.5 * mx] or sm
        return {"sm_mhz": float(np.median(busy)) if busy else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


ALU_PEAK_TFLOPS = None                # set in main() once the device is known (74.45 on B200)


def layer_costs(L, hbm_gbs):
    """Algorithmic flops / bytes of one layer and its roofline time (us)."""
    es = 2 if L.dtype == "f16" else 4
    flops = 2.0 * L.nonzero_macs
    P = len(L.patterns)
    byts = (L.N * L.C * L.H * L.W * es + L.N * L.F * L.H * L.W * es + L.K * (4 * es + 2)
            + L.F * (4 * (P + 1) + 8) + 4 * L.F)
    t_alu = flops / (ALU_PEAK_TFLOPS * 1e12) * 1e6
    t_hbm = byts / (hbm_gbs * 1e9) * 1e6
    return flops, byts, max(t_alu, t_hbm), ("alu" if t_alu >= t_hbm else "hbm")


def executed_tensor_flops(L, plan):
    """16-bit MMA flops the dense tensor-core kernel issues for a layer (0 for the CUDA-core kernels)."""
    if plan["variant"] != 4:
        return 0.0
    taps = 1 if 9 * L.C <= 64 else 9          # tiny C: neighbourhood gathered into the channel dimension
    cp = 64 if taps == 1 else (L.C + 63) // 64 * 64
    bn = plan["filters_per_warp"]
    fp = (L.F + bn - 1) // bn * bn
    ftiles = fp // bn
    ctas = plan["grid_y"] if plan["grid_y"] > 1 else plan["grid_x"]     # persistent kernels report their tile count in grid_y
    rows = ctas // (ftiles * max(plan["channel_splits"], 1)) * max(128, plan["tile_rows"] * plan["tile_cols"])
    terms = 1 if L.dtype == "f16" else 3
    return terms * 2.0 * taps * cp * fp * rows


class VggStack:
    def __init__(self, N: int, B, synth, torch):
        self.N, self.B, self.torch = N, B, torch
        self.layers = [synth.vgg16_layer(i, N=N) for i in range(13)]
        self.handles = [B.encode(L.weights, L.mask, L.patterns, N=N, H=L.H, W=L.W, relu=True, bias=L.bias)
                        for L in self.layers]
        self.pools = [1 if i in synth.VGG16_POOL_AFTER else 0 for i in range(13)]
        self.stack = B.Stack(self.handles, self.pools)
        self.out_shape = self.stack.out_shape()
        self.x_host = synth.vgg16_input(N)

    def per_layer_buffers(self):
        """Device tensors so that each layer can be timed alone on realistic (post-ReLU-like) inputs."""
        torch = self.torch
        bufs = []
        g = torch.Generator(device="cuda").manual_seed(7)
        for L in self.layers:
            x = torch.rand((self.N, L.C, L.H, L.W), device="cuda", generator=g)
            y = torch.empty((self.N, L.F, L.H, L.W), device="cuda")
            bufs.append((x, y))
        return bufs


def oracle_stack_pass(synth, oracle, layers, x, keep=None):
    """One pass of the CPU oracle over the 13 chained layers (pools included); returns seconds.  keep: a list that
    receives the final activations."""
    t0 = time.perf_counter()
    cur = x
    for i, L in enumerate(layers):
        cur = oracle.conv3x3(cur, L.weights, L.mask, L.bias, True)
        if i in synth.VGG16_POOL_AFTER:
            cur = oracle.maxpool2x2(cur)
    dt = time.perf_counter() - t0
    if keep is not None:
        keep.append(cur)
    return dt


def parity_against_oracle(synth, gpu_outputs):
    """Part of the CPU-baseline leg: the oracle chained over single images of the benchmark input, compared with what
    the timed stacks produced for them.  gpu_outputs: {batch: (image indices, float32 array [len, F, H, W])}.
    Ratios are in units of the single-layer tolerance 1e-4 * max(|o|, rms(o)); a 13-layer chain is allowed sqrt(13)."""
    import oracle
    layers = [synth.vgg16_layer(i, N=1) for i in range(13)]
    out = {"tolerance": "|gpu - oracle| <= 1e-4 * max(|o|, rms(o)) per layer; sqrt(13) of that for the 13-layer chain",
           "allowed_ratio": round(13 ** 0.5, 3), "checked": []}
    worst_all = 0.0
    for batch, (imgs, got) in gpu_outputs.items():
        x = synth.vgg16_input(batch)
        for j, n in enumerate(imgs):
            keep = []
            oracle_stack_pass(synth, oracle, layers, np.ascontiguousarray(x[n:n + 1]), keep)
            ref = keep[0][0].astype(np.float64)
            g = got[j].astype(np.float64)
            rms = float(np.sqrt(np.mean(ref * ref)))
            ratio = float((np.abs(g - ref) / (1e-4 * np.maximum(np.abs(ref), rms))).max()) if np.all(np.isfinite(g)) else float("inf")
            out["checked"].append({"batch": batch, "image": int(n), "worst_ratio": round(ratio, 3)})
            worst_all = max(worst_all, ratio)
    out["worst_ratio"] = round(worst_all, 3)
    out["ok"] = bool(worst_all <= 13 ** 0.5)
    return out


def time_oracle_sample(synth, seconds_hint=12.0):
    """CPU oracle on a bounded sample of the workload: the whole 13-layer stack on ONE image (the benchmark step has 32),
    repeated for about seconds_hint seconds."""
    import oracle
    layers = [synth.vgg16_layer(i, N=1) for i in range(13)]
    x = synth.vgg16_input(1)
    oracle.conv3x3(x[:, :, :8, :8], layers[0].weights, layers[0].mask, layers[0].bias, True)   # load outside the timing
    tot, reps = 0.0, 0
    while tot < seconds_hint and reps < 200:
        tot += oracle_stack_pass(synth, oracle, layers, x)
        reps += 1
    dt = tot / reps
    flops = sum(2.0 * L.nonzero_macs for L in layers)
    cores = oracle.num_threads()
    oracle.set_num_threads(1)                                    # the same sample on one core, two passes
    try:
        dt1 = min(oracle_stack_pass(synth, oracle, layers, x) for _ in range(2))
    finally:
        oracle.set_num_threads(cores)
    return {"value": flops / dt / 1e9, "unit": "GFLOP/s", "cores": cores, "kind": "oracle",
            "single_thread_value": flops / dt1 / 1e9,
            "sample": f"the 13-layer stack on one image (1/32 of a benchmark step), {reps} passes, {dt * 1e3:.0f} ms each, "
                      f"OpenMP over filters; single_thread_value = the same pass on one core ({dt1 * 1e3:.0f} ms)"}


def time_layer(h, x, y, stream, torch, reps=20, flush=None):
    """Mean time (us) of one layer call, CUDA events on the launching stream.  Small cases (flush given) replay the call
    as a one-node-chain CUDA graph: launching from Python costs more than such a layer runs."""
    for _ in range(3):
        h.conv(x, y, stream)
    torch.cuda.synchronize()
    graph = None
    if flush is not None:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            h.conv(x, y, torch.cuda.current_stream().cuda_stream)
        graph.replay()
        torch.cuda.synchronize()
    tot = 0.0
    for _ in range(reps):
        if flush is not None:
            flush.fill_(1.0)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        if graph is not None:
            graph.replay()
        else:
            h.conv(x, y, stream)
        b.record()
        torch.cuda.synchronize()
        tot += a.elapsed_time(b)
    return tot / reps * 1e3


def run_suite(args):
    """The other configurations of the baseline as a table (one JSON object per line on stdout):
    config 2, the ResNet-50-shaped fp16 layers, the pattern-count x connectivity sweep (with the filter reorder on and
    with a seeded random filter order), and the ablation ladder no-opt -> +reorder -> tiled -> tensor cores."""
    import torch
    from paper_2001_00138_b200 import build as lib_build, binding as B, synth
    lib_build.build_library()
    B.load()
    peaks, _ = measured_peaks()
    hbm = float(peaks["hbm_gbs"])
    global ALU_PEAK_TFLOPS
    ALU_PEAK_TFLOPS = alu_peak_tflops(torch)
    stream = torch.cuda.current_stream().cuda_stream
    flush = torch.empty(256 * 1024 * 1024 // 4, device="cuda")
    variants = {"auto": 0, "noopt": 1, "reorder": 2, "tiled": 3, "dense_tc": 4, "pattern_run": 5}

    def measure(tag, L, N, variant="auto", order=None, reps=20):
        dt = B.F16 if L.dtype == "f16" else B.F32
        tdt = torch.float16 if L.dtype == "f16" else torch.float32
        try:
            h = B.encode(L.weights, L.mask, L.patterns, N=N, H=L.H, W=L.W, dtype=dt, relu=True, bias=L.bias,
                         order=order, variant=variants[variant])
        except B.PatdnnError as e:
            print(json.dumps({"suite": tag, "layer": L.name, "batch": N, "variant": variant, "error": str(e)}))
            return
        x = torch.rand((N, L.C, L.H, L.W), device="cuda").to(tdt)
        y = torch.empty((N, L.F, L.H, L.W), device="cuda", dtype=tdt)
        small = x.numel() * x.element_size() + y.numel() * y.element_size() < 128 * 2**20
        us = time_layer(h, x, y, stream, torch, reps=reps, flush=flush if small else None)
        L.N = N
        flops, byts, roof_us, bound = layer_costs(L, hbm)
        plan = h.plan()
        print(json.dumps({"suite": tag, "layer": L.name, "batch": N, "variant": variant,
                          "kernel": "generated_fp32" if plan.get("generated") else
                                    {1: "noopt", 2: "reorder", 3: "tiled", 4: "dense_tc", 5: "pattern_run"}[plan["variant"]],
                          "filter_order": "random" if order is not None else "fkr", "K": L.K,
                          "us": round(us, 2), "gflops_nonzero": round(flops / us / 1e3, 1),
                          "roofline_us": round(roof_us, 2), "bound": bound, "frac": round(roof_us / us, 3),
                          "lane_use": round(L.K / plan["entries"], 3) if plan["variant"] == 5 else None,
                          "l2": "flushed between launches" if small else "working set larger than L2"}), flush=True)
        h.free()

    which = args.suite.split(",")
    if "cfg2" in which or "all" in which:
        measure("config2", synth.config2(draw_input=False), 1)
    if "resnet" in which or "all" in which:
        for i in range(4):
            for N in (1, 32):
                measure("resnet50_fp16", synth.resnet50_layer(i, N=N, draw_input=False), N)
    if "sweep" in which or "all" in which:
        for npat in synth.SWEEP_PATTERNS:
            for prune in synth.SWEEP_PRUNE:
                L = synth.sweep_layer(npat, prune, N=64, draw_input=False)
                measure("sweep", L, 64)
                measure("sweep", L, 64, order=synth.random_filter_order(512, 7))
                measure("sweep", L, 64, variant="tiled")
                measure("sweep", L, 64, variant="tiled", order=synth.random_filter_order(512, 7))
                measure("sweep", L, 64, variant="pattern_run")
                measure("sweep", L, 64, variant="pattern_run", order=synth.random_filter_order(512, 7))
    if "crossover" in which or "all" in which:
        # beyond the baseline's sweep: where the kernel whose time follows the kept kernels overtakes the dense tensor-core path
        for npat in (4, 8, 12):
            for prune in (0.95, 0.97, 0.99):
                L = synth.make_layer(f"sweep_p{npat}_prune{int(prune * 100)}", F=512, C=512, N=64, H=14, W=14, seed=5100 + npat,
                                     n_patterns=npat, prune=prune, draw_input=False)
                for variant in ("auto", "dense_tc", "pattern_run"):
                    measure("crossover", L, 64, variant=variant)
                measure("crossover", L, 64, variant="pattern_run", order=synth.random_filter_order(512, 7))
    if "cifar" in which or "all" in which:
        suite_cifar_stack(B, synth, torch, hbm, stream)
    if "storage" in which or "all" in which:
        suite_storage(B, synth)
    if "context" in which or "all" in which:
        suite_dense_context(synth, torch)
    if "ablation" in which or "all" in which:
        seen = set()
        for i in range(13):
            if synth.VGG16_CONVS[i] in seen:
                continue
            seen.add(synth.VGG16_CONVS[i])
            L = synth.vgg16_layer(i, N=1)
            for variant in ("noopt", "reorder", "tiled", "dense_tc"):
                measure("ablation_vgg_unique_layers", L, 1, variant=variant, reps=5 if variant in ("noopt", "reorder") else 20)


def suite_cifar_stack(B, synth, torch, hbm, stream):
    """VGG-16's conv stack on a CIFAR-sized 32x32 input (the paper's second dataset): 32,32,16,16,8,8,8,4,4,4,2,2,2."""
    for N in (1, 32, 256):
        layers = [synth.vgg16_layer(i, N=N, spatial_scale=7) for i in range(13)]
        handles = [B.encode(L.weights, L.mask, L.patterns, N=N, H=L.H, W=L.W, relu=True, bias=L.bias) for L in layers]
        pools = [1 if i in synth.VGG16_POOL_AFTER else 0 for i in range(13)]
        stack = B.Stack(handles, pools)
        x = torch.from_numpy(synth.vgg16_input(N, 7)).cuda()
        out = torch.empty(stack.out_shape(), device="cuda")
        graph = torch.cuda.CUDAGraph()
        stack.run(x, out, stream)
        torch.cuda.synchronize()
        with torch.cuda.graph(graph):
            stack.run(x, out, torch.cuda.current_stream().cuda_stream)
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 20
        a.record()
        for _ in range(reps):
            graph.replay()
        b.record()
        torch.cuda.synchronize()
        us = a.elapsed_time(b) / reps * 1e3
        for h in handles:
            h.check()
        costs = [layer_costs(L, hbm) for L in layers]
        flops, roof = sum(c[0] for c in costs), sum(c[2] for c in costs)
        print(json.dumps({"suite": "cifar_vgg16_stack", "batch": N, "us": round(us, 1),
                          "gflops_nonzero": round(flops / us / 1e3, 1), "roofline_us": round(roof, 1),
                          "frac": round(roof / us, 3),
                          "kernels": "".join("j" if h.plan().get("generated") else {3: "t", 4: "D"}.get(h.plan()["variant"], "g")
                                             for h in handles),
                          "timing": "CUDA-graph replay of the chained stack, working set L2-resident"}), flush=True)
        stack.free()
        for h in handles:
            h.free()


def suite_storage(B, synth):
    """Index and total bytes of the FKW arrays against CSR over the same weights (Section 6.4's comparison), from the
    arrays the encoder really emits; overall rates 8x / 12x / 18x = 4-of-9 patterns times connectivity pruning."""
    for rate in (8, 12, 18):
        keep = 9.0 / (4.0 * rate)
        for (C, F) in ((256, 256), (512, 512)):
            L = synth.make_layer(f"storage_c{C}f{F}_{rate}x", F=F, C=C, N=1, H=14, W=14, seed=6000 + rate, n_patterns=8,
                                 prune=1.0 - keep, draw_input=False)
            h = B.encode(L.weights, L.mask, L.patterns, N=1, H=14, W=14, host_only=True)
            a = h.export()
            K = int(a["index"].shape[0])
            nnz = 4 * K
            fkw_idx32 = 4 * (a["offset"].size + a["reorder"].size + a["index"].size + a["stride"].size)
            fkw_idx16 = 2 * a["index"].size + 4 * a["offset"].size + 2 * a["reorder"].size + 2 * a["stride"].size
            fkw_idx8 = 1 * a["index"].size + 2 * (a["offset"].size + a["reorder"].size + a["stride"].size)
            csr_idx32 = 4 * (F + 1) + 4 * nnz
            csr_idx16 = 4 * (F + 1) + 2 * nnz
            w_bytes = 4 * nnz
            print(json.dumps({"suite": "storage_fkw_vs_csr", "layer": L.name, "overall_rate": rate, "kernels_kept": K,
                              "weights_bytes": w_bytes, "fkw_index_bytes_i32": fkw_idx32, "csr_index_bytes_i32": csr_idx32,
                              "fkw_index_bytes_u16": fkw_idx16, "csr_index_bytes_u16": csr_idx16,
                              "index_saving_i32": round(1 - fkw_idx32 / csr_idx32, 4),
                              "total_saving_i32": round(1 - (fkw_idx32 + w_bytes) / (csr_idx32 + w_bytes), 4),
                              "total_saving_u16": round(1 - (fkw_idx16 + w_bytes) / (csr_idx16 + w_bytes), 4),
                              # the widths that fit the paper's 93.4 % / 46.7 %: one byte per index[] entry, two per
                              # per-filter entry, against four bytes per CSR column index
                              "index_saving_u8_vs_csr_i32": round(1 - fkw_idx8 / csr_idx32, 4),
                              "total_saving_u8_vs_csr_i32": round(1 - (fkw_idx8 + w_bytes) / (csr_idx32 + w_bytes), 4)}), flush=True)
            h.free()


def suite_dense_context(synth, torch):
    """Library context, not a target: torch's dense conv2d (cuDNN, fp32 without TF32) on the unpruned shape of each
    unique VGG layer, next to which the pattern-sparse numbers of the headline run can be read."""
    import torch.nn.functional as Fn
    torch.backends.cudnn.allow_tf32 = False
    torch.backends.cuda.matmul.allow_tf32 = False
    flush = torch.empty(256 * 1024 * 1024 // 4, device="cuda")
    for N in (1, 32):
        seen = set()
        for i in range(13):
            if synth.VGG16_CONVS[i] in seen:
                continue
            seen.add(synth.VGG16_CONVS[i])
            C, F, S = synth.VGG16_CONVS[i]
            x = torch.rand((N, C, S, S), device="cuda")
            w = torch.randn((F, C, 3, 3), device="cuda") * 0.05
            for _ in range(3):
                Fn.conv2d(x, w, padding=1)
            torch.cuda.synchronize()
            tot, reps = 0.0, 10
            for _ in range(reps):
                if N == 1:
                    flush.fill_(1.0)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                Fn.conv2d(x, w, padding=1)
                b.record()
                torch.cuda.synchronize()
                tot += a.elapsed_time(b)
            us = tot / reps * 1e3
            print(json.dumps({"suite": "dense_conv2d_context", "layer": f"c{C}f{F}_{S}", "batch": N, "us": round(us, 1),
                              "dense_gflops": round(2.0 * 9 * C * F * S * S * N / us / 1e3, 1),
                              "library": "torch.nn.functional.conv2d (cuDNN), fp32, TF32 off"}), flush=True)


def workload_config(batch: int) -> dict:
    """The `config` object of the JSON line: the workload both arms are quoted on."""
    return {"workload": f"vgg16_3x3_stack_n{batch}", "batch_per_gpu": batch, "layers": 13,
            "patterns": 8, "connectivity_pruning": "0% layer 1, 60% layers 2-13",
            "l2": ("working set larger than L2 (first activation alone is %d MB); input buffers rotated"
                   % (batch * 64 * 224 * 224 * 4 // 2**20)) if batch >= 8 else "see batch1 leg",
            "step": "13 conv layers chained by the library: RGB layer as FP32 code generated for it, 12 tensor-core GEMM "
                    "layers (some with a K-split tail launch), every kernel writing the next layer's operands directly; "
                    "the 4 max-pools are taken in epilogues"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2001_00138_b200 import synth
    import oracle
    oracle.build()
    layers = [synth.vgg16_layer(i, N=1) for i in range(13)]
    x = synth.vgg16_input(1)
    for _ in range(max(min(args.warmup, 2), 1)):
        oracle_stack_pass(synth, oracle, layers, x)
    dt = sum(oracle_stack_pass(synth, oracle, layers, x) for _ in range(args.steps)) / args.steps
    val = sum(2.0 * L.nonzero_macs for L in layers) / dt / 1e9
    sample = "each step = the 13-layer stack on one image (1/32 of the GPU arm's step) on the host cores"
    print(json.dumps({
        "impl": "reference", "metric": "effective GFLOP/s on nonzero MACs, pattern-sparse 3x3 conv", "value": val,
        "unit": "GFLOP/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(args.batch),            # the GPU arm's configuration; what one step samples of it: `sample`
        "cpu_baseline": {"value": val, "unit": "GFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": val, "unit": "GFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=32)
    ap.add_argument("--no-extras", action="store_true", help="skip the batch-1 and CPU-baseline legs")
    ap.add_argument("--suite", default="", help="instead of the headline step: cfg2,resnet,sweep,ablation,cifar,storage,context or all "
                                                "(one JSON line per measured point); also: crossover")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.suite:
        run_suite(args)
        return
    args.warmup = max(args.warmup, 3)

    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    from paper_2001_00138_b200 import build as lib_build
    if rank == 0:
        lib_build.build_library()
    if world > 1:
        dist.barrier()
    from paper_2001_00138_b200 import binding as B, synth
    B.load()
    peaks, peak_kind = measured_peaks()
    hbm = float(peaks["hbm_gbs"])
    stream = torch.cuda.current_stream().cuda_stream
    global ALU_PEAK_TFLOPS
    ALU_PEAK_TFLOPS = alu_peak_tflops(torch)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def bench_stack(N, steps, warmup, flush_l2):
        vs = VggStack(N, B, synth, torch)
        costs = [layer_costs(L, hbm) for L in vs.layers]
        flops = sum(c[0] for c in costs)
        nbuf = 3
        xs = [torch.from_numpy(vs.x_host).cuda() for _ in range(nbuf)]
        out = torch.empty(vs.out_shape, device="cuda")
        flush = torch.empty(256 * 1024 * 1024 // 4, device="cuda") if flush_l2 else None
        for i in range(warmup):
            vs.stack.run(xs[i % nbuf], out, stream)
        barrier()
        # (1) whole-step timing: K steps between one pair of events (per-step events when L2 is flushed in between)
        B.reset_launch_count()
        sampler = ClockSampler(local_rank)
        sampler.start()
        barrier()
        if flush is None:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(steps):
                vs.stack.run(xs[i % nbuf], out, stream)
            e1.record()
            barrier()
            total_ms = e0.elapsed_time(e1)
        else:
            evs = []
            for i in range(steps):
                flush.fill_(float(i))
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                vs.stack.run(xs[i % nbuf], out, stream)
                b.record()
                evs.append((a, b))
            barrier()
            total_ms = sum(a.elapsed_time(b) for a, b in evs)
        launches = B.launch_count()
        clocks = sampler.stop()
        # what the timed steps produced for the first and the last image (checked against the oracle in the CPU leg)
        vs.stack.run(xs[0], out, stream)
        torch.cuda.synchronize()
        imgs = sorted({0, N - 1})
        kept_out = (imgs, out[imgs].cpu().numpy())
        # (1a) per-layer times INSIDE the chained step: events between the layers' launches (a separate pass)
        in_step = np.zeros(13)
        tsteps = max(3, min(steps, 10))
        for i in range(tsteps):
            if flush is not None:
                flush.fill_(float(i))
            in_step += vs.stack.run_timed(xs[i % nbuf], out, stream).astype(np.float64)
        in_step = in_step / tsteps * 1e3                      # us
        # (1b) the same step as one CUDA-graph replay (launch overhead off the critical path)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            vs.stack.run(xs[0], out, torch.cuda.current_stream().cuda_stream)
        graph.replay()
        torch.cuda.synchronize()
        gevs = []
        for i in range(steps):
            if flush is not None:
                flush.fill_(float(i))
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            graph.replay()
            b.record()
            gevs.append((a, b))
        torch.cuda.synchronize()
        graph_ms = sum(a.elapsed_time(b) for a, b in gevs) / steps
        del graph
        # (2) per-layer timing of the conv kernel alone (same stream, events around each launch)
        bufs = vs.per_layer_buffers()
        for (x, y), h in zip(bufs, vs.handles):
            h.conv(x, y, stream)
        torch.cuda.synchronize()
        reps = max(3, min(steps, 10))
        layer_ms = [0.0] * 13
        # small batch: a launch from Python costs more than the kernels run, so each layer is replayed as a one-call graph
        graphs = None
        if flush is not None:
            graphs = []
            for (x, y), h in zip(bufs, vs.handles):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    h.conv(x, y, torch.cuda.current_stream().cuda_stream)
                graphs.append(g)
            torch.cuda.synchronize()
        for _ in range(reps):
            evs = []
            for li, ((x, y), h) in enumerate(zip(bufs, vs.handles)):
                if flush is not None:
                    flush.fill_(1.0)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                if graphs is not None:
                    graphs[li].replay()
                else:
                    h.conv(x, y, stream)
                b.record()
                evs.append((a, b))
            torch.cuda.synchronize()
            for i, (a, b) in enumerate(evs):
                layer_ms[i] += a.elapsed_time(b) / reps
        del graphs
        del bufs
        # (3) end to end through the host-buffer entry point: pinned input -> device -> stack -> pinned output
        xh = torch.from_numpy(vs.x_host).pin_memory()
        oh = torch.empty(vs.out_shape, dtype=torch.float32).pin_memory()
        vs.stack.run_host(xh.numpy(), oh.numpy(), stream)
        barrier()
        e2e_steps = max(3, min(steps, 10))
        t0 = time.perf_counter()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(e2e_steps):
            vs.stack.run_host(xh.numpy(), oh.numpy(), stream)
        e1.record()
        torch.cuda.synchronize()
        e2e_blocking_ms = max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3) / e2e_steps
        # the same through the pipelined entry point: a stream of batches, two in flight, every batch's copy-in and
        # copy-out inside the timed region (wall clock: the work spans three streams)
        xh2 = [xh, torch.from_numpy(vs.x_host).pin_memory()]
        oh2 = [oh, torch.empty(vs.out_shape, dtype=torch.float32).pin_memory()]
        vs.stack.submit_host(xh2[0].numpy(), oh2[0].numpy(), stream)
        vs.stack.wait_host()
        barrier()
        pipe_steps = max(6, min(steps, 20))
        t0 = time.perf_counter()
        for i in range(pipe_steps):
            if i >= 2:
                vs.stack.wait_host()
            vs.stack.submit_host(xh2[i & 1].numpy(), oh2[i & 1].numpy(), stream)
        vs.stack.wait_host()
        vs.stack.wait_host()
        torch.cuda.synchronize()
        e2e_ms = (time.perf_counter() - t0) * 1e3 / pipe_steps
        res = {
            "ms_per_step": total_ms / steps, "graph_ms_per_step": graph_ms, "flops": flops, "launches": launches, "clocks": clocks,
            "layer_us": [m * 1e3 for m in layer_ms], "in_step_us": [float(v) for v in in_step], "kept_out": kept_out, "costs": costs, "e2e_ms": e2e_ms, "e2e_blocking_ms": e2e_blocking_ms,
            "h2d": int(xh.numel() * 4), "d2h": int(oh.numel() * 4),
            "plans": [h.plan() for h in vs.handles], "names": [L.name for L in vs.layers],
            "layer_objs": vs.layers,
        }
        vs.stack.free()
        for h in vs.handles:
            h.free()
        return res

    r = bench_stack(args.batch, args.steps, args.warmup, flush_l2=False)
    ms = r["ms_per_step"]
    e2e_ms = r["e2e_ms"]
    from paper_2001_00138_b200 import replicas
    ms, e2e_ms = replicas.max_over_ranks([ms, e2e_ms], device="cuda")     # the slowest replica sets the time
    roof_us = sum(c[2] for c in r["costs"])
    bytes_step = sum(c[1] for c in r["costs"])
    achieved = r["flops"] / (ms * 1e-3) / 1e12                            # kept-weight TFLOP/s of the timed step
    n_alu = sum(1 for c in r["costs"] if c[3] == "alu")

    def tensor_pipe(res, step_ms):
        """Executed 16-bit MMA flops of the tensor-core layers over their time INSIDE the chained step."""
        tc = [(executed_tensor_flops(L, p), u) for L, p, u in zip(res["layer_objs"], res["plans"], res["in_step_us"])]
        fl = sum(f for f, _ in tc)
        us = sum(u for f, u in tc if f > 0)
        capped = "sw_power_cap" in (res["clocks"].get("reasons") or [])
        burst = float(peaks.get("bf16_tflops", 1590.0))
        sustained = float(peaks.get("bf16_tflops_sustained", burst))
        peak = sustained if capped else burst
        ach = fl / (us * 1e-6) / 1e12 if us > 0 else 0.0
        return {"bound": "tensor", "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": ach / peak,
                "peak_source": f"{peak_kind} bf16 cuBLAS peak, " + ("sustained figure: the power cap was active during the timed region"
                                                                   if capped else "burst figure: the timed region is short and ran at "
                                                                   "full clocks with no power cap"),
                "executed_flops_per_step": fl, "us_per_step": us, "launches_per_step": sum(1 for f, _ in tc if f > 0),
                "step_us": step_ms * 1e3,
                "what": "tcgen05 implicit GEMM kernels (bf16 hi/lo split, three products per fp32 product, zero-padded "
                        "dense work): executed MMA flops / summed in-step time of the tensor-core layers, measured with "
                        "events between the layers of the chained stack (patdnn_stack_run_timed)"}

    line = {
        "metric": "effective GFLOP/s on nonzero MACs, pattern-sparse 3x3 conv",
        "value": replicas.whole_job_value(r["flops"], ms * 1e-3, world) / 1e9,
        "unit": "GFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(args.batch),
        "clocks": r["clocks"],
        "e2e": {"value": world * r["flops"] / (e2e_ms * 1e-3) / 1e9, "unit": "GFLOP/s",
                "h2d_bytes_per_step": r["h2d"], "d2h_bytes_per_step": r["d2h"], "ms_per_step": e2e_ms,
                "blocking_ms_per_step": r["e2e_blocking_ms"],
                "how": "patdnn_stack_submit_host / wait_host: pinned host input -> device -> 13 layers -> pinned host output for "
                       "every step, two steps in flight (copies of one step overlap the kernels of the other); "
                       "blocking_ms_per_step = the same through patdnn_stack_run_host, one step at a time"},
        "gpu_launches": int(r["launches"]), "graph_ms_per_step": r["graph_ms_per_step"],
        # The roofline of the metric: kept-weight flops at the FP32 CUDA-core peak against algorithmic bytes at the
        # measured HBM bandwidth, per layer the slower of the two, summed over the step and divided by the step time.
        "roofline": {"bound": "alu", "achieved": achieved, "peak": ALU_PEAK_TFLOPS, "unit": "TFLOP/s",
                     "frac": roof_us / (ms * 1e3), "traffic": TRAFFIC_BYTES_PER_LAUNCH, "traffic_note": TRAFFIC_NOTE,
                     "definition": "per layer max(2 * nonzero MACs / FP32 CUDA-core peak, algorithmic bytes / measured HBM "
                                   "bandwidth); frac = sum over the 13 layers / ms_per_step (whole chained step, fused pools "
                                   "included); achieved = kept-weight flops of the step / ms_per_step",
                     "peak_source": "derived: SMs x 128 FP32 lanes x 2 flop x max SM clock (an FFMA-chain probe measured 71.6)",
                     "frac_alu_only": achieved / ALU_PEAK_TFLOPS, "roofline_us_per_step": roof_us,
                     "flops_per_step": r["flops"], "algorithmic_bytes_per_step": bytes_step,
                     "layers_alu_bound": n_alu, "layers_hbm_bound": 13 - n_alu,
                     "hbm_peak_gbs": hbm, "hbm_peak_kind": peak_kind},
        "tensor_pipe": tensor_pipe(r, ms),
        "layers": [{"name": n, "in_step_us": round(iu, 2), "standalone_us": round(u, 2), "roofline_us": round(c[2], 2),
                    "bound": c[3], "frac_in_step": round(c[2] / iu, 3) if iu > 0 else None, "frac_standalone": round(c[2] / u, 3),
                    "kernel": "generated_fp32" if p.get("generated") else {3: "tiled", 4: "dense_tc"}.get(p["variant"], "generic"),
                    "tile": f"{p['tile_rows']}x{p['tile_cols']}x{p['filters_per_warp']}f", "grid": p["grid_x"]}
                   for n, u, iu, c, p in zip(r["names"], r["layer_us"], r["in_step_us"], r["costs"], r["plans"])],
        "layers_note": "in_step_us: the layer's kernels inside the chained step (events between layers); standalone_us: "
                       "the layer called alone through patdnn_conv, NCHW in and out (layout kernel included)",
    }
    if rank == 0 and world == 1 and not args.no_extras:
        r1 = bench_stack(1, max(args.steps, 20), args.warmup, flush_l2=True)
        roof1 = sum(c[2] for c in r1["costs"])
        line["batch1"] = {"workload": "vgg16_3x3_stack_n1", "ms_per_step": r1["ms_per_step"],
                          "graph_ms_per_step": r1["graph_ms_per_step"],
                          "value": r1["flops"] / (r1["ms_per_step"] * 1e-3) / 1e9, "unit": "GFLOP/s",
                          "l2": "256 MB buffer written between timed steps",
                          "roofline": {"bound": "alu", "achieved": r1["flops"] / (r1["ms_per_step"] * 1e-3) / 1e12,
                                       "peak": ALU_PEAK_TFLOPS, "unit": "TFLOP/s",
                                       "frac": roof1 / (r1["ms_per_step"] * 1e3),
                                       "frac_graph_replay": roof1 / (r1["graph_ms_per_step"] * 1e3),
                                       "roofline_us_per_step": roof1},
                          "tensor_pipe": tensor_pipe(r1, r1["ms_per_step"]),
                          "in_step_us": [round(u, 2) for u in r1["in_step_us"]],
                          "standalone_us": [round(u, 2) for u in r1["layer_us"]],
                          "e2e_ms": r1["e2e_ms"], "gpu_launches": int(r1["launches"])}
        import oracle
        oracle.build()
        line["cpu_baseline"] = time_oracle_sample(synth)
        line["parity"] = parity_against_oracle(synth, {args.batch: r["kept_out"], 1: r1["kept_out"]})
    elif rank == 0:
        line["cpu_baseline"] = None
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
