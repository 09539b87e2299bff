"""Synchronous data-parallel optimiser step on top of the lazy-tensor library.

The paper trains data-parallel by summing gradients across replicas with the compiler's cross-replica-sum
(Section 4, "distributed training"; Section 5.3 scales ResNet-50 that way).  Here the exchange is an all-reduce
of `torch.distributed` (NCCL over NVLink on GPUs, gloo on CPU for tests) and everything else is the traced
graph: gradients live in one flat buffer, cut into buckets that follow the order in which the multi-tensor Adam
kernel walks the tensors; each bucket is summed on a side stream while the next one is being issued; the
averaging (1 / world size) is a run-time scalar of the traced Adam graph, so the update stays one fused
multi-tensor launch that is recorded once and replayed.

Only argument marshalling and stream plumbing happen here; no arithmetic on tensor values.
"""
from __future__ import annotations

import math

import numpy as np


class DataParallelAdam:
    """Parameters, gradients and Adam moments of `shapes` in four flat f32 buffers, and the step that
    all-reduces the gradient buffer bucket by bucket and applies one traced Adam update."""

    ALIGN = 64  # elements: every tensor starts on a 256-byte boundary of its flat buffer

    def __init__(self, ctx, shapes, *, bucket_bytes: int = 25 << 20, lr: float = 1e-3, beta1: float = 0.9,
                 beta2: float = 0.999, eps: float = 1e-8, process_group=None):
        import torch
        import torch.distributed as dist

        self.ctx = ctx
        self.shapes = [tuple(s) for s in shapes]
        self.hyper = dict(lr=lr, beta1=beta1, beta2=beta2, eps=eps)
        self.group = process_group
        self.world = dist.get_world_size(process_group) if dist.is_available() and dist.is_initialized() else 1
        self.dry = ctx.device < 0
        dev = torch.device("cpu") if self.dry else torch.device("cuda", ctx.device)
        sizes = [int(np.prod(s)) for s in self.shapes]
        self.offsets, total = [], 0
        for n in sizes:
            self.offsets.append(total)
            total += (n + self.ALIGN - 1) // self.ALIGN * self.ALIGN
        self.sizes, self.total = sizes, total
        self.flat = {k: torch.zeros(total, dtype=torch.float32, device=dev) for k in ("p", "g", "m", "v")}
        self.tensors = {k: [ctx.from_device_ptr(self.flat[k].data_ptr() + 4 * off, "f32", shp, keep=self.flat[k])
                            for off, shp in zip(self.offsets, self.shapes)] for k in self.flat}
        # buckets: consecutive tensors, in launch order, of at least bucket_bytes of gradient each
        self.buckets, lo = [], 0
        for i in range(len(sizes)):
            end = self.offsets[i] + (sizes[i] + self.ALIGN - 1) // self.ALIGN * self.ALIGN
            if 4 * (end - lo) >= bucket_bytes or i == len(sizes) - 1:
                self.buckets.append((lo, end))
                lo = end
        self.step_count = 0
        self._scalars = None
        self._inv_world = None
        self._side = None if self.dry else torch.cuda.Stream(device=dev)

    def view(self, which: str, i: int):
        """Torch view of tensor i of the flat buffer `which` ("p", "g", "m" or "v")."""
        return self.flat[which][self.offsets[i]:self.offsets[i] + self.sizes[i]].view(self.shapes[i])

    def all_reduce_gradients(self) -> None:
        """Sums the gradient buffer over the ranks, one all-reduce per bucket, on a side stream; the stream the
        context launches on waits for the last of them."""
        if self.world == 1:
            return
        import torch
        import torch.distributed as dist

        g = self.flat["g"]
        if self.dry:
            for lo, hi in self.buckets:
                dist.all_reduce(g[lo:hi], op=dist.ReduceOp.SUM, group=self.group)
            return
        main = torch.cuda.ExternalStream(self.ctx.stream) if self.ctx.stream else torch.cuda.default_stream(g.device)
        self._side.wait_stream(main)  # the gradients were produced on the main stream
        with torch.cuda.stream(self._side):
            for lo, hi in self.buckets:
                dist.all_reduce(g[lo:hi], op=dist.ReduceOp.SUM, group=self.group)
        main.wait_stream(self._side)

    def _record(self) -> None:
        from workloads import traces  # the traced Adam program is shared with the benchmark configurations

        ctx = self.ctx
        self._scalars = traces.AdamScalars(ctx, step=self.step_count, **self.hyper)
        self._inv_world = ctx.scalar(1.0 / self.world, dynamic=True)  # run-time slot: one program for any world size
        t = self.tensors
        for p, g, m, v in zip(t["p"], t["g"], t["m"], t["v"]):
            traces.adam_update(ctx, p, ctx.op("mul", g, self._inv_world), m, v, self._scalars)
        ctx.barrier()

    def step(self) -> None:
        """All-reduce, then one Adam update of every tensor (recorded on the first call, replayed afterwards)."""
        self.step_count += 1
        self.all_reduce_gradients()
        if self._scalars is None:
            self._record()
            return
        h, t = self.hyper, self.step_count
        self.ctx.scalar_set(self._scalars.sqrt_bc2, math.sqrt(1.0 - h["beta2"] ** t))
        self.ctx.scalar_set(self._scalars.step_size, h["lr"] / (1.0 - h["beta1"] ** t))
        self.ctx.replay()
