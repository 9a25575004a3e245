"""Runs one of the synthetic workloads through the library a fixed number of times.

    python -m paper_1901_05350_b200.run_workload --workload mobilenet224 --batch 128 --steps 3
    python -m paper_1901_05350_b200.run_workload --workload matmul --size 4096 --steps 3
    python -m paper_1901_05350_b200.run_workload --workload block --batch 32 --steps 3
    python -m paper_1901_05350_b200.run_workload --workload depthwise --batch 128 --hw 14 --channels 512 --stride 1
    python -m paper_1901_05350_b200.run_workload --workload pointwise --batch 128 --hw 14 --channels 512 --cout 512
    python -m paper_1901_05350_b200.run_workload --workload maxpool --batch 128 --hw 112 --channels 64 --stride 2
    python -m paper_1901_05350_b200.run_workload --workload add --batch 128 --hw 56 --channels 128
    python -m paper_1901_05350_b200.run_workload --workload batch_matmul --batch 16 --size 1024
    python -m paper_1901_05350_b200.run_workload --workload mobilenet224 --batch 128 --math bf16 --per-layer
    python -m paper_1901_05350_b200.run_workload --workload matmul_bf16 --m 25088 --k 512 --n 512

A plain driver for profilers and quick timing: it builds the inputs, runs `--warmup` untimed and
`--steps` timed passes on one stream, prints the mean device time per pass, and exits.
"""
from __future__ import annotations

import argparse
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", choices=["mobilenet224", "mobilenet128_025", "matmul", "block", "depthwise", "pointwise", "maxpool", "add",
                             "batch_matmul", "matmul_bf16"],
                    default="mobilenet224")
    ap.add_argument("--batch", type=int, default=128)
    ap.add_argument("--size", type=int, default=512, help="matmul: M = K = N")
    ap.add_argument("--hw", type=int, default=112, help="depthwise / pointwise: input height = width")
    ap.add_argument("--channels", type=int, default=32, help="depthwise / pointwise: input channels")
    ap.add_argument("--cout", type=int, default=64, help="pointwise: output channels")
    ap.add_argument("--stride", type=int, default=1, help="depthwise / maxpool: stride")
    ap.add_argument("--dilation", type=int, default=1, help="depthwise: dilation (with stride 1)")
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=1)
    ap.add_argument("--math", choices=["tf32", "fp32", "bf16"], default="tf32",
                    help="bf16: the narrow-storage mode (models only)")
    ap.add_argument("--m", type=int, default=25088, help="matmul_bf16: rows of A")
    ap.add_argument("--k", type=int, default=512, help="matmul_bf16: inner dimension")
    ap.add_argument("--n", type=int, default=512, help="matmul_bf16: rows of Bt")
    ap.add_argument("--per-layer", action="store_true", help="model workloads: print every layer's mean device time")
    args = ap.parse_args()

    import torch

    import paper_1901_05350_b200 as tfjsb
    import seeded_inputs as si

    ctx = tfjsb.Context(0, math=args.math)
    if args.workload == "matmul":
        a, b = si.config_matmul(args.size)
        a, b = torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda()
        out = torch.empty(args.size, args.size, device="cuda")
        step = lambda: ctx.matmul(a, b, out=out)
    elif args.workload == "matmul_bf16":
        a = torch.from_numpy(si.uniform(7, 0, (args.m, args.k), -1.0, 1.0)).cuda().to(torch.bfloat16)
        bt = torch.from_numpy(si.uniform(7, 1, (args.n, args.k), -1.0, 1.0)).cuda().to(torch.bfloat16)
        out = torch.empty(args.m, args.n, dtype=torch.bfloat16, device="cuda")
        step = lambda: ctx.matmul_bf16(a, bt, out=out)
    elif args.workload == "block":
        x, (dw, pw) = si.config_separable_block(batch=args.batch)
        x = torch.from_numpy(x).cuda()
        wd, bd = torch.from_numpy(dw.filter).cuda(), torch.from_numpy(dw.bias).cuda()
        wp, bp = torch.from_numpy(pw.filter).cuda(), torch.from_numpy(pw.bias).cuda()
        mid = torch.empty(x.shape, device="cuda")
        out = torch.empty(x.shape[:3] + (pw.out_channels,), device="cuda")

        def step():
            ctx.depthwise_conv2d(x, wd, dw.strides, dw.pad, dw.dilations, bd, dw.act, out=mid)
            ctx.conv2d(mid, wp, pw.strides, pw.pad, pw.dilations, bp, pw.act, out=out)
    elif args.workload == "batch_matmul":
        a = torch.from_numpy(si.uniform(7, 0, (args.batch, args.size, args.size), -1.0, 1.0)).cuda()
        b = torch.from_numpy(si.uniform(7, 1, (args.batch, args.size, args.size), -1.0, 1.0)).cuda()
        out = torch.empty(args.batch, args.size, args.size, device="cuda")
        step = lambda: ctx.batch_matmul(a, b, False, True, out=out)  # b given K-contiguous: no transpose pass
    elif args.workload in ("maxpool", "add"):
        x = torch.from_numpy(si.uniform(7, 0, (args.batch, args.hw, args.hw, args.channels), -1.0, 1.0)).cuda()
        if args.workload == "maxpool":
            strides = (args.stride, args.stride)
            out = ctx.max_pool(x, (3, 3), strides, "same")
            step = lambda: ctx.max_pool(x, (3, 3), strides, "same", out=out)
        else:
            y = torch.from_numpy(si.uniform(7, 1, x.shape, -1.0, 1.0)).cuda()
            out = torch.empty_like(x)
            step = lambda: ctx.binary("add", x, y, out=out)
        print(f"{args.workload}: {x.numel() * 4 / 1e6:.1f} MB in per operand, {out.numel() * 4 / 1e6:.1f} MB out")
    elif args.workload in ("depthwise", "pointwise"):
        x = torch.from_numpy(si.uniform(7, 0, (args.batch, args.hw, args.hw, args.channels), 0.0, 6.0)).cuda()
        if args.workload == "depthwise":
            w = torch.from_numpy(si.normal(7, 1, (3, 3, args.channels, 1), 0.0, 0.47)).cuda()
            b = torch.from_numpy(si.normal(7, 2, (args.channels,), 0.0, 0.01)).cuda()
            strides, dil = (args.stride, args.stride), (args.dilation, args.dilation)
            out = ctx.depthwise_conv2d(x, w, strides, "same", dil, b, "relu6")
            step = lambda: ctx.depthwise_conv2d(x, w, strides, "same", dil, b, "relu6", out=out)
        else:
            from seeded_inputs.workloads import Layer

            layer = Layer("conv2d", (1, 1), (1, 1), (1, 1), "same", "relu6", args.cout, "pw")
            si.make_model_weights([layer], args.channels, 7)
            model = ctx.model([layer], x.shape)  # the executor keeps the weights K-contiguous
            out = torch.empty(model.output_shape, device="cuda")
            step = lambda: model.run(x, out=out)
    else:
        alpha, hw = (1.0, 224) if args.workload == "mobilenet224" else (0.25, 128)
        x, layers = si.config_mobilenet(alpha, hw, args.batch, seed=si.CONFIG_SEEDS["mobilenet_100_224"])
        model = ctx.model(layers, x.shape)
        x = torch.from_numpy(x).cuda()
        out = torch.empty(model.output_shape, device="cuda")
        step = lambda: model.run(x, out=out)
        if args.per_layer:
            model.run(x, out=out)
            for name, ms in zip(model.layer_names, model.profile(x, out=out, reps=max(args.steps, 1))):
                print(f"  {name:12s} {ms * 1e3:8.2f} us")

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(args.steps):
        step()
    stop.record()
    torch.cuda.synchronize()
    ctx.check_device_status()
    print(f"{args.workload}: {start.elapsed_time(stop) / max(args.steps, 1):.4f} ms per pass over {args.steps} passes")
    return 0


if __name__ == "__main__":
    sys.exit(main())
