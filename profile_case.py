"""Runs one synthetic layer a few times through the C ABI -- the small case to put under ``ncu``.

    python profile_case.py --layer vgg6 --batch 4 --reps 3 [--variant tiled]

Layers: ``cfg1``, ``cfg2``, ``vggK`` (K = 1..13, VGG-16-shaped layer K), ``resnetK`` (K = 1..4, fp16),
``sweep:P:PRUNE`` (512->512 @14x14), ``custom:F:C:H:W:P:PRUNE``.  ``--chain M`` (vggK only) runs layers K .. K+M-1 as a
stack, so that the in-stack kernels (first layer writing the next layer's operands, fused pools) can be captured.
Prints the mean launch time measured with CUDA events.
"""
from __future__ import annotations

import argparse
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))


def make(layer: str, batch: int):
    from paper_2001_00138_b200 import synth
    if layer == "cfg1":
        return synth.config1()
    if layer == "cfg2":
        return synth.config2(draw_input=False)
    if layer.startswith("vgg"):
        return synth.vgg16_layer(int(layer[3:]) - 1, N=batch)
    if layer.startswith("resnet"):
        return synth.resnet50_layer(int(layer[6:]) - 1, N=batch, draw_input=False)
    if layer.startswith("sweep:"):
        _, p, prune = layer.split(":")
        return synth.sweep_layer(int(p), float(prune), N=batch, draw_input=False)
    if layer.startswith("custom:"):                       # custom:F:C:H:W:P:PRUNE
        _, F, C, H, W, P, prune = layer.split(":")
        return synth.make_layer(layer, F=int(F), C=int(C), N=batch, H=int(H), W=int(W), seed=1, n_patterns=int(P),
                                prune=float(prune), draw_input=False)
    raise SystemExit(f"unknown layer {layer}")


def run_chain(args, torch, B):
    from paper_2001_00138_b200 import synth
    first = int(args.layer[3:]) - 1
    idx = list(range(first, first + args.chain))
    layers = [synth.vgg16_layer(i, N=args.batch) for i in idx]
    handles = [B.encode(L.weights, L.mask, L.patterns, N=args.batch, H=L.H, W=L.W, relu=True, bias=L.bias) for L in layers]
    stack = B.Stack(handles, [1 if i in synth.VGG16_POOL_AFTER else 0 for i in idx])
    L0 = layers[0]
    x = torch.rand((args.batch, L0.C, L0.H, L0.W), device="cuda")
    y = torch.empty(stack.out_shape(), device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    stack.run(x, y, st)
    torch.cuda.synchronize()
    tot = None
    for _ in range(args.reps):
        ms = stack.run_timed(x, y, st)
        tot = ms if tot is None else tot + ms
    print(f"stack of {[L.name for L in layers]} N={args.batch}: per-layer us {[round(float(v) * 1e3 / args.reps, 1) for v in tot]}")
    stack.free()
    for h in handles:
        h.free()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layer", default="vgg6")
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--variant", default="auto", choices=["auto", "noopt", "reorder", "tiled", "dense", "prun"])
    ap.add_argument("--chain", type=int, default=1)
    args = ap.parse_args()
    import torch
    from paper_2001_00138_b200 import binding as B, build
    build.build_library()
    if args.chain > 1:
        run_chain(args, torch, B)
        return
    L = make(args.layer, args.batch)
    N = L.N if args.layer in ("cfg1", "cfg2") else args.batch
    dt = B.F16 if L.dtype == "f16" else B.F32
    tdt = torch.float16 if L.dtype == "f16" else torch.float32
    variant = {"auto": 0, "noopt": 1, "reorder": 2, "tiled": 3, "dense": 4, "prun": 5}[args.variant]
    h = B.encode(L.weights, L.mask, L.patterns, N=N, H=L.H, W=L.W, dtype=dt, relu=True, bias=L.bias, variant=variant)
    x = torch.rand((N, L.C, L.H, L.W), device="cuda").to(tdt)
    y = torch.empty((N, L.F, L.H, L.W), device="cuda", dtype=tdt)
    st = torch.cuda.current_stream().cuda_stream
    h.conv(x, y, st)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.reps):
        h.conv(x, y, st)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / args.reps
    flops = 2.0 * 4 * L.K * L.H * L.W * N
    print(f"{L.name} N={N} K={L.K} plan={h.plan()}")
    print(f"mean launch {us:.1f} us, {flops / us / 1e6:.2f} TFLOP/s on kept weights")
    h.free()


if __name__ == "__main__":
    main()
