"""Run one convolution layer through the C ABI a few times and print its plan and timing.

    python -m paper_1606_00094_b200.run_layer --layer conv2 [--batch 20] [--reps 20] [--tile -1] [--split 0]
                                               [--variant auto|direct|k1conv|tconv] [--math auto|fp32|tf32]

Layers: cfg1..cfg4 (the single-layer benchmark configurations) and conv1..conv5 (the layers of the
AlexNet-shaped stack).  Handy for profiling one kernel in isolation (e.g. under ncu) and for trying tiles.
"""
from __future__ import annotations

import argparse

import torch

from . import binding as B
from . import workloads as wl


def layer_shape(name: str, batch: int) -> wl.ConvShape:
    if name.startswith("cfg"):
        s = wl.CONFIGS[int(name[3:])].shape
        return wl.ConvShape(batch or s.N, s.C, s.H, s.W, s.K, s.R, s.S, s.stride, s.pad, s.relu)
    convs = [op.shape for op in wl.alexnet_stack(batch or 20) if op.kind == "conv"]
    return convs[int(name[4:]) - 1]


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--layer", default="conv2")
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--tile", type=int, default=-1)
    ap.add_argument("--split", type=int, default=0)
    ap.add_argument("--tune", type=int, default=0)
    ap.add_argument("--variant", default="auto", choices=["auto", "direct", "k1conv", "tconv"])
    ap.add_argument("--math", default="auto", choices=["auto", "fp32", "tf32", "tf32x3"])
    args = ap.parse_args()
    s = layer_shape(args.layer, args.batch)
    variant = {"auto": -1, "direct": 0, "k1conv": 1, "tconv": 2}[args.variant]
    math = {"auto": 0, "fp32": 1, "tf32": 2, "tf32x3": 3}[args.math]
    plan = B.ConvPlan(s.as_tuple(), math=math, variant=variant, tile_id=args.tile, split_k=args.split, tune=args.tune)
    x = torch.from_numpy(wl.half_normal(1, (s.N, s.C, s.H, s.W))).cuda()
    w = torch.from_numpy(wl.normal(2, (s.K, s.C, s.R, s.S), 0.0, (2.0 / (s.C * s.R * s.S)) ** 0.5)).cuda()
    b = torch.from_numpy(wl.normal(3, (s.K,), 0.0, 0.01)).cuda()
    out = torch.empty(plan.out_shape, dtype=torch.float32, device="cuda")
    plan.bind_filters(w)
    for _ in range(3):
        plan(x, w, b, out=out)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.reps):
        plan(x, w, b, out=out)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.reps
    status = B.boda_query_status()
    print(f"{args.layer} {s.as_tuple()}: {plan.describe()}")
    print(f"  {ms * 1e3:.2f} us per call ({args.reps} back-to-back calls, staging included), "
          f"{s.flops / ms / 1e9:.1f} TFLOP/s, device status {status}")
    plan.close()


if __name__ == "__main__":
    main()
