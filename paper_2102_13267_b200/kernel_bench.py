"""Kernel-only timing of the benchmark configurations and of the common fusion groups (also the driver for ncu captures).

    python -m paper_2102_13267_b200.kernel_bench [c1,c2,c2p,c3,c4,c5,idioms,long,reduce,reduced] [--iters N] [--sets K] [key=value ...]

For each configuration: traces the graph and flushes it `iters` times over rotating buffer sets (larger than L2
together), queued behind a busy stream so that the GPU, not the host, sets the pace.  Two figures are printed:
every launch between its own two CUDA events (`lt_set_kernel_timing`), and "back to back": one pair of events around
all the launches, kernel timing off (for C5 the steps are replayed, the host cannot record 161 tensors that fast).
`key=value` pairs are context options (e.g. fusion=0, compiled=0, ieee=1, debug.waves=2).  With `--iters 4 --sets 1` it is the
small workload used for `ncu --set full` captures.
"""
from __future__ import annotations

import argparse
import math
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

import torch

import paper_2102_13267_b200 as lt
from workloads import configs, traces
from workloads.resnet50 import parameter_shapes


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("configs", nargs="?", default="c1,c2,c2p,c3,c4,c5")
    ap.add_argument("--iters", type=int, default=40)
    ap.add_argument("--sets", type=int, default=0, help="buffer sets to rotate through (0 = enough for 1 GB)")
    ap.add_argument("--long-shapes", default="8192x16384,2048x65536", help="rows x columns of the `long` case")
    ap.add_argument("--only", default="", help="of the idioms / long / reduce cases, run those whose name contains this")
    ap.add_argument("options", nargs="*")
    args = ap.parse_args()
    which = args.configs.split(",")
    opts = dict(kv.split("=") for kv in args.options)
    dev = torch.device("cuda", 0)

    def context():
        ctx = lt.LazyContext(device=0)
        for k, v in opts.items():
            ctx.set_option(k, int(v))
        return ctx

    def bf16(shape, std=1.0):
        return (torch.randn(shape, device=dev) * std).to(torch.bfloat16)

    def hold_gpu(ms=4.0):
        """Keeps the stream busy for a few milliseconds so that the flushes recorded next queue up behind it and
        then run back to back: the per-launch event brackets then hold kernel time, not the host's pace."""
        torch.cuda._sleep(int(ms * 1e-3 * 1.9e9))

    def report(name, nbytes, kt, region_ms=None):
        ms = sum(v["ms"] for v in kt.values()) / args.iters
        n = sum(v["launches"] for v in kt.values()) / args.iters
        tail = ""
        if region_ms is not None:  # the same flushes without per-launch events: one pair of events around all of them
            r = region_ms / args.iters
            tail = f"  | back to back {1e3 * r:7.1f} us/flush {nbytes / r / 1e6:8.1f} GB/s"
        print(f"{name:18s} {1e3 * ms:9.1f} us/flush {nbytes / ms / 1e6:8.1f} GB/s  {n:.0f} launches/flush{tail}", flush=True)

    def back_to_back(flush_all):
        """Milliseconds for all iterations queued behind a busy stream, between two events, kernel timing off."""
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        hold_gpu()
        e0.record()
        flush_all()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    def run(name, cfg, make, trace):
        nbytes = configs.algorithmic_bytes(cfg)
        nsets = args.sets or max(2, math.ceil(1.2e9 / nbytes))
        ctx = context()
        sets = [make(ctx) for _ in range(nsets)]
        keep = [None] * nsets
        for i in range(nsets + 2):  # every set flushed once: no allocator call is left for the timed flushes
            keep[i % nsets] = trace(ctx, sets[i % nsets])
            ctx.barrier()
        torch.cuda.synchronize()
        ctx.set_kernel_timing(True)
        ctx.kernel_timing()
        hold_gpu()
        for i in range(args.iters):
            keep[i % nsets] = trace(ctx, sets[i % nsets])
            ctx.barrier()
        kt = ctx.kernel_timing()
        ctx.set_kernel_timing(False)

        def flush_all():
            for i in range(args.iters):
                keep[i % nsets] = trace(ctx, sets[i % nsets])
                ctx.barrier()

        region = back_to_back(flush_all) if args.iters >= 20 else None
        report(name, nbytes, kt, region)
        del keep, sets
        ctx.close()

    if "c1" in which:
        shape = configs.FULL["c1"]
        run("c1", "c1", lambda c: [c.from_torch(torch.rand(shape, device=dev) * 2 - 1) for _ in range(4)],
            lambda c, s: traces.elementwise_chain(c, *s))
    for name, prim in (("c2", False), ("c2p", True)):
        if name in which:
            shape = configs.FULL["c2"]
            run(name, "c2", lambda c: (c.from_torch(bf16(shape)), c.from_torch(bf16(shape)), c.from_torch(bf16((shape[1],), 0.02))),
                lambda c, s, prim=prim: traces.mlp_epilogue(c, *s, primitive_gelu=prim))
    if "c3" in which:
        shape = configs.FULL["c3"]
        run("c3", "c3", lambda c: (c.from_torch(bf16(shape)), c.from_torch(bf16(shape)),
                                   c.from_torch(1 + 0.02 * torch.randn(shape[1], device=dev)),
                                   c.from_torch(0.02 * torch.randn(shape[1], device=dev))),
            lambda c, s: traces.residual_dropout_layernorm(c, *s, shape=shape, p=0.1, eps=1e-5, seed=1, offset=0))
    if "c4" in which:
        shape = configs.FULL["c4"]
        run("c4", "c4", lambda c: (c.from_torch(bf16(shape, 4.0)),),
            lambda c, s: traces.causal_softmax(c, *s, shape=shape, scale=1 / math.sqrt(128)))
    # common fusion groups (workloads/idioms.py) on [16384 x 1024]: name, bytes per element moved
    from workloads import idioms

    ishape = (16384, 1024)
    for name, kinds, trace in idioms.ALL:
        if name not in which and "idioms" not in which:
            continue
        per_elem = sum((2 if k.endswith("bf16") else 4) for k in kinds if k.startswith("mat")) + (4 if name.endswith("f32") else 2)
        nbytes = per_elem * ishape[0] * ishape[1]

        def make(c, kinds=kinds):
            out = []
            for k in kinds:
                shp = ishape if k.startswith("mat") else (ishape[1],)
                t = torch.randn(shp, device=dev)
                out.append(c.from_torch(t.to(torch.bfloat16) if k.endswith("bf16") else t))
            return out

        nsets = args.sets or max(2, math.ceil(1.2e9 / nbytes))
        ctx = context()
        sets = [make(ctx) for _ in range(nsets)]
        keep = [None] * nsets
        for i in range(nsets + 2):
            keep[i % nsets] = trace(ctx, sets[i % nsets], ishape[1])
            ctx.barrier()
        torch.cuda.synchronize()
        ctx.set_kernel_timing(True)
        ctx.kernel_timing()
        hold_gpu()
        for i in range(args.iters):
            keep[i % nsets] = trace(ctx, sets[i % nsets], ishape[1])
            ctx.barrier()
        kt = ctx.kernel_timing()
        ctx.set_kernel_timing(False)

        def flush_all():
            for i in range(args.iters):
                keep[i % nsets] = trace(ctx, sets[i % nsets], ishape[1])
                ctx.barrier()

        region = back_to_back(flush_all) if args.iters >= 20 else None
        report(name[:18], nbytes, kt, region)
        del keep, sets
        ctx.close()
    # rows longer than a thread group's registers (fused long-row kernels), and reductions over columns / everything
    def generic(name, nbytes, make, trace):
        if args.only and args.only not in name:
            return
        nsets = args.sets or max(2, math.ceil(1.2e9 / nbytes))
        ctx = context()
        sets = [make(ctx) for _ in range(nsets)]
        keep = [None] * nsets
        for i in range(nsets + 2):
            keep[i % nsets] = trace(ctx, sets[i % nsets])
            ctx.barrier()
        torch.cuda.synchronize()
        ctx.set_kernel_timing(True)
        ctx.kernel_timing()
        hold_gpu()
        for i in range(args.iters):
            keep[i % nsets] = trace(ctx, sets[i % nsets])
            ctx.barrier()
        kt = ctx.kernel_timing()
        ctx.set_kernel_timing(False)

        def flush_all():
            for i in range(args.iters):
                keep[i % nsets] = trace(ctx, sets[i % nsets])
                ctx.barrier()

        region = back_to_back(flush_all) if args.iters >= 20 else None
        report(name[:18], nbytes, kt, region)
        del keep, sets
        ctx.close()

    if "long" in which:
        for rows, cols in (tuple(int(v) for v in sh.split("x")) for sh in args.long_shapes.split(",")):
            for iname in ("softmax_bf16", "layernorm_bf16", "softmax_f32", "layernorm_f32"):
                _, kinds, trace = next(e for e in idioms.ALL if e[0] == iname)
                es = 4 if iname.endswith("f32") else 2

                def make(c, kinds=kinds, rows=rows, cols=cols):
                    out = []
                    for k in kinds:
                        t = torch.randn((rows, cols) if k.startswith("mat") else (cols,), device=dev)
                        out.append(c.from_torch(t.to(torch.bfloat16) if k.endswith("bf16") else t))
                    return out

                generic(f"{iname} {cols}", 2 * es * rows * cols, make, lambda c, s_, trace=trace, cols=cols: trace(c, s_, cols))
    if "reduce" in which:
        for rows, cols in ((16384, 4096), (1 << 20, 64)):
            for op in ("col_sum", "all_sum", "row_sum"):
                generic(f"{op} {rows}x{cols}", 4 * rows * cols, lambda c, rows=rows, cols=cols: [c.from_torch(torch.randn((rows, cols), device=dev))],
                        lambda c, s_, op=op: c.op(op, s_[0]))
        generic("row_sum 4096x65536", 4 * 4096 * 65536, lambda c: [c.from_torch(torch.randn((4096, 65536), device=dev))],
                lambda c, s_: c.op("row_sum", s_[0]))
        # reductions of a computed value, (a - b)^2: the two inputs are all that has to move (run with specialise=1 to have
        # the fused kernel from the first flush, specialise=0 for the unfused plan)
        for op in ("col_sum", "all_sum"):
            for dt, es in (("f32", 4), ("bf16", 2)):
                def make(c, dt=dt):
                    ts = [torch.randn((16384, 4096), device=dev) for _ in range(2)]
                    return [c.from_torch(t.to(torch.bfloat16) if dt == "bf16" else t) for t in ts]

                def trace(c, s_, op=op):
                    d = c.op("sub", s_[0], s_[1])
                    return c.op(op, c.op("mul", d, d))

                generic(f"{op} (a-b)^2 {dt}", 2 * es * 16384 * 4096, make, trace)
    if "reduced" in which:  # reductions of computed values (workloads/idioms.py REDUCED) on [16384 x 4096]: inputs are all that moves
        for iname, kinds, trace in idioms.REDUCED:
            nbytes = sum((2 if k.endswith("bf16") else 4) * 16384 * 4096 for k in kinds)

            def make(c, kinds=kinds):
                out = []
                for k in kinds:
                    t = torch.randn((16384, 4096), device=dev)
                    out.append(c.from_torch(t.to(torch.bfloat16) if k.endswith("bf16") else t))
                return out

            generic(iname, nbytes, make, lambda c, s_, trace=trace: trace(c, s_, 4096))
    if "c5" in which:
        shapes = parameter_shapes()
        ctx = context()
        P, G, M, V = ([ctx.from_torch(torch.randn(s, device=dev) * 0.05) for s in shapes] for _ in range(4))
        step = 0
        for _ in range(min(3, args.iters)):
            step += 1
            traces.adam_step(ctx, P, G, M, V, step=step)
            ctx.barrier()
        torch.cuda.synchronize()
        ctx.set_kernel_timing(True)
        ctx.kernel_timing()
        for _ in range(args.iters):
            hold_gpu(8.0)  # recording a step of 161 tensors takes the host a few milliseconds
            step += 1
            traces.adam_step(ctx, P, G, M, V, step=step)
            ctx.barrier()
        kt = ctx.kernel_timing()
        ctx.set_kernel_timing(False)
        # back to back: the host cannot record 161 tensors as fast as the kernel runs, so the steps are replayed
        s = traces.AdamScalars(ctx, step=step + 1)
        for p, g, m, v in zip(P, G, M, V):
            traces.adam_update(ctx, p, g, m, v, s)
        ctx.barrier()
        region = back_to_back(lambda: [ctx.replay() for _ in range(args.iters)]) if args.iters >= 20 else None
        report("c5", configs.algorithmic_bytes("c5"), kt, region)
        ctx.close()


if __name__ == "__main__":
    main()
