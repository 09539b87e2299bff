#!/usr/bin/env python
"""Benchmark of the fused-graph executor.

A step is one pass of the whole path over one batch: trace the MLP-epilogue graph
(out = x + GELU_tanh(h + bias), bf16 [8192 x 4096], fp32 arithmetic), barrier (canonicalise,
hash, cache lookup, bind, launch), with the inputs already resident in HBM.  The metric is
HBM GB/s = algorithmic bytes (each input read once, the output written once) / time.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank runs the same
per-GPU workload on its own buffers -- the path has no exchange step -- and the value is the
sum over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "fused-graph HBM GB/s"
UNIT = "GB/s"
WORKLOAD = "c2_mlp_epilogue_bf16_8192x4096"
SHAPE = (8192, 4096)
N_SETS = 6  # rotating input/output sets: 6 x 201 MB > L2 (126 MB), so every step streams from HBM
FALLBACK_HBM_GBS = 6650.0

_SAMPLER = r"""
import sys, time
import pynvml as nv
nv.nvmlInit()
h = nv.nvmlDeviceGetHandleByIndex(int(sys.argv[1]))
mx = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
def sample():
    try:
        r = nv.nvmlDeviceGetCurrentClocksEventReasons(h)
    except Exception:
        r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(h)
    return time.time(), nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM), int(r)
sample()  # the first query of each kind can take a long time: get it over with before reporting ready
print("max", mx, flush=True)
while True:
    print(*sample(), flush=True)
    time.sleep(0.0005)
"""

_REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
            0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x10: "sync_boost",
            0x100: "display_clock_setting"}


class ClockSampler:
    """Reads SM clock and throttle reasons (read-only NVML queries) from a child process."""

    def __init__(self, device_index: int):
        self.proc = None
        self.head = ""
        try:
            self.proc = subprocess.Popen([sys.executable, "-c", _SAMPLER, str(device_index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.head = self.proc.stdout.readline()  # "max <MHz>": from here on the child is sampling
        except Exception:
            self.proc = None

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.02)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        mx, inside, all_ = None, [], []
        for ln in (self.head + out).splitlines():
            p = ln.split()
            if len(p) == 2 and p[0] == "max":
                mx = float(p[1])
            elif len(p) == 3:
                rec = (float(p[0]), float(p[1]), int(p[2]))
                all_.append(rec)
                if t0 <= rec[0] <= t1:
                    inside.append(rec)
        use = inside or all_[-3:]
        reasons = set()
        for _, _, r in use:
            for bit, name in _REASONS.items():
                if r & bit:
                    reasons.add(name)
        return {"sm_mhz": statistics.median([c for _, c, _ in use]) if use else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(inside)}


def measured_peak() -> tuple[float, str]:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, STREAM-style copy)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (earlier measurement on this pool)"


# DRAM bytes of one launch of the dominant kernel on this workload, from the ncu capture summarised in
# profiles/lt_c_ew_c2_mlp_epilogue.md, with the hash of the kernel sources it was taken on.
NCU_TRAFFIC = {"bytes": 164452352, "sources_sha256": "cb37d535b0589e4e748f62b9f0da8b2a694ec4c816d62f5e7b07da8d98e18b30"}
KERNEL_SOURCES = ("paper_2102_13267_b200/csrc/compiled.cu", "paper_2102_13267_b200/csrc/compiled_shells.cuh",
                  "paper_2102_13267_b200/csrc/compiled_programs.inc", "paper_2102_13267_b200/csrc/vm_ops.cuh",
                  "paper_2102_13267_b200/csrc/vm.h", "paper_2102_13267_b200/csrc/pdl.cuh")


def kernel_sources_sha256() -> str:
    h = hashlib.sha256()
    for rel in KERNEL_SOURCES:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def ncu_traffic() -> float | None:
    """Measured DRAM bytes per launch, or None once the kernel sources differ from the profiled ones."""
    try:
        return float(NCU_TRAFFIC["bytes"]) if kernel_sources_sha256() == NCU_TRAFFIC["sources_sha256"] else None
    except Exception:
        return None


# --------------------------------------------------------------------------- oracle arm
class OracleRun:
    """The CPU eager oracle (one op at a time, as it stands) on the first `rows` rows of the workload."""

    def __init__(self, rows: int, threads: int):
        from oracle import eager
        from workloads import configs

        eager.set_threads(threads)
        x, h, b = configs.c2_inputs(0, (rows, SHAPE[1]))
        self.O = eager.EagerOracle()
        self.leaves = (self.O.leaf(x, "bf16"), self.O.leaf(h, "bf16"), self.O.leaf(b, "bf16"))
        self.rows = rows
        self.nbytes = configs.algorithmic_bytes("c2", (rows, SHAPE[1]))

    def step(self) -> float:
        from workloads import traces

        t0 = time.perf_counter()
        traces.mlp_epilogue(self.O, *self.leaves, primitive_gelu=False)
        return time.perf_counter() - t0


def cpu_baseline(budget_s: float = 12.0) -> dict:
    from oracle import eager

    threads = eager.max_threads()
    probe = OracleRun(256, threads)
    probe.step()
    t_row = probe.step() / 256
    rows = int(min(SHAPE[0], max(256, budget_s / max(t_row, 1e-9))))
    run = OracleRun(rows, threads)
    run.step()
    passes = int(max(1, min(50, budget_s / max(t_row * rows, 1e-6))))
    sec = sum(run.step() for _ in range(passes))
    return {"value": run.nbytes * passes / sec / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{rows} of {SHAPE[0]} rows of the workload, {passes} passes, {sec:.2f} s, OpenMP over elements"}


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import eager

    threads = eager.max_threads()
    probe = OracleRun(256, threads)
    probe.step()
    t_row = probe.step() / 256
    total = max(1, args.steps + args.warmup)
    rows = int(max(1, min(SHAPE[0], 90.0 / total / max(t_row, 1e-9))))
    run = OracleRun(rows, threads)
    for _ in range(args.warmup):
        run.step()
    sec = sum(run.step() for _ in range(args.steps))
    value = run.nbytes * args.steps / sec / 1e9
    sample = f"each step: {rows} of {SHAPE[0]} rows of the workload through the CPU eager oracle"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * sec / max(args.steps, 1), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "trace": "convert x3, add, gelu_tanh, add, convert", "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------------------ our arm
def max_over_ranks(ms: float, world: int, device=None) -> float:
    """Slowest rank's time: the replicas share no data, so the job's time is the maximum."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist

    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_gbs(bytes_per_rank_step: int, steps: int, world: int, ms: float) -> float:
    """Whole-job GB/s: every rank moved bytes_per_rank_step per step, in the slowest rank's time."""
    return world * bytes_per_rank_step * steps / (ms / 1e3) / 1e9


def run_ours(args) -> None:
    import torch
    import torch.distributed as dist

    import paper_2102_13267_b200 as lt
    from workloads import configs, traces

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    ctx = lt.LazyContext(device=local)
    nbytes = configs.algorithmic_bytes("c2", SHAPE)

    # seeded synthetic inputs: one host draw per rank, shifted copies for the other sets
    x, h, b = configs.c2_inputs(1000 + rank, SHAPE)
    tx = torch.from_numpy(x.view(np.int16)).to(dev).view(torch.bfloat16)
    th = torch.from_numpy(h.view(np.int16)).to(dev).view(torch.bfloat16)
    tb = torch.from_numpy(b.view(np.int16)).to(dev).view(torch.bfloat16)
    sets = []
    for s in range(N_SETS):
        xs = torch.roll(tx, shifts=s, dims=0).contiguous() if s else tx
        hs = torch.roll(th, shifts=-s, dims=0).contiguous() if s else th
        sets.append((ctx.from_torch(xs), ctx.from_torch(hs), ctx.from_torch(tb.clone())))
    outs = [None] * N_SETS

    def step(i: int, primitive: bool = False) -> None:
        X, H, Bv = sets[i % N_SETS]
        outs[i % N_SETS] = traces.mlp_epilogue(ctx, X, H, Bv, primitive_gelu=primitive)
        ctx.barrier()

    def sync_all() -> None:
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def timed(n_steps: int, fn) -> float:
        sync_all()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(n_steps):
            fn(i)
        e1.record()
        torch.cuda.synchronize()
        return max_over_ranks(e0.elapsed_time(e1), world, dev)

    # Every rotating set is flushed before anything is timed, whatever --warmup says: the first flush on a set
    # obtains its output block from the allocator (a cudaMalloc of 64 MiB takes milliseconds), later ones reuse
    # the block the context's pool got back when the previous output of that set was dropped.
    for i in range(N_SETS + 2):
        step(i)
    for i in range(max(args.warmup, 3)):
        step(i)
    sampler = ClockSampler(local) if rank == 0 else None
    sync_all()
    ctx.reset_stats()
    host_s = [0.0]

    def timed_steps(n_steps: int) -> float:
        """Exactly n_steps steps between two events.  A short spin kernel ahead of the first event lets the host
        get a few steps ahead, as it is in the steady state of a long run, so that a 20-step region is not
        dominated by the first launch's latency; the spin itself ends before the first event is recorded."""
        sync_all()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda._sleep(int(1.0e-3 * 1.9e9))
        e0.record()
        n_host = min(n_steps, 200)  # the host's own pace: taken while the launch queue cannot be full yet
        h0 = time.perf_counter()
        for i in range(n_host):
            step(i)
        host_s[0] = (time.perf_counter() - h0) / max(n_host, 1)
        for i in range(n_host, n_steps):
            step(i)
        e1.record()
        torch.cuda.synchronize()
        return max_over_ranks(e0.elapsed_time(e1), world, dev)

    w0 = time.time()
    ms = timed_steps(args.steps)
    st = ctx.stats()
    host_us_per_step = 1e6 * host_s[0]
    value = aggregate_gbs(nbytes, args.steps, world, ms)
    ms_local = ms  # (max over ranks; at one GPU this rank's own time)
    # second pass with every launch bracketed by its own pair of events (costs ~2 us per step on the stream);
    # long enough (>= 2000 launches of the same kernel on the same buffers) for the clock sampler to see the load
    ctx.set_kernel_timing(True)
    ctx.kernel_timing()
    timed(max(min(args.steps, 4000), 2000), step)
    kt = ctx.kernel_timing()
    ctx.set_kernel_timing(False)
    w1 = time.time()
    clocks = sampler.stop(w0, w1) if sampler else None
    if clocks is not None:
        clocks["window"] = "timed region + the bracketed pass that follows it (same kernel, same buffers)"

    # ---- end to end through the C ABI with host buffers: H2D of the inputs and D2H of the result every step
    e2e_steps = max(3, min(args.steps, 30))
    pin = [torch.from_numpy(a.view(np.int16)).pin_memory() for a in (x, h, b)]
    host_out = torch.empty(SHAPE, dtype=torch.int16).pin_memory()

    # Two contexts on two streams, used alternately (what a caller does to keep both directions of the host link
    # busy): step i's inputs go up and its kernel is queued on one stream, then the result of step i-1 is read
    # back on the other -- lt_fetch blocks the host only for that read.  Every step's inputs are copied from pinned
    # host memory and every step's result is read into pinned host memory inside the timed region.
    streams = [torch.cuda.Stream(device=dev) for _ in range(2)]
    ectx = [lt.LazyContext(device=local, stream=st.cuda_stream) for st in streams]
    host_outs = [host_out, torch.empty(SHAPE, dtype=torch.int16).pin_memory()]
    in_flight = [None, None]

    def e2e_submit(k: int) -> None:
        c = ectx[k]
        X = c.from_host(pin[0].numpy().view(np.uint16), "bf16")
        H = c.from_host(pin[1].numpy().view(np.uint16), "bf16")
        Bv = c.from_host(pin[2].numpy().view(np.uint16), "bf16")
        in_flight[k] = traces.mlp_epilogue(c, X, H, Bv, primitive_gelu=False)
        c.barrier()

    def e2e_collect(k: int) -> None:
        if in_flight[k] is not None:
            ectx[k].fetch_into(in_flight[k], host_outs[k].data_ptr(), host_outs[k].numel() * 2)
            in_flight[k] = None

    def e2e_step(i: int) -> None:
        e2e_submit(i % 2)
        e2e_collect((i + 1) % 2)

    def e2e_run(n: int) -> None:
        for i in range(n):
            e2e_step(i)
        e2e_collect((n + 1) % 2)  # the last step's result

    e2e_run(3)
    sync_all()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    e2e_run(e2e_steps)  # returns when the last result is in host memory
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), world, dev)
    for c in ectx:
        c.close()
    e2e_value = aggregate_gbs(nbytes, e2e_steps, world, e2e_ms)

    dp_adam = None if args.no_extra else data_parallel_adam(lt, torch, local, world)  # collective: every rank takes part
    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel: algorithmic bytes per launch / average launch duration
    peak, peak_src = measured_peak()
    # The timed region holds nothing but this kernel's launches, one per step, queued back to back (the host
    # records and flushes a step faster than the kernel runs), so region time / launches is the kernel's
    # average launch duration including the gap to the next launch.  The per-launch brackets of the second
    # pass are reported beside it; they add the cost of two event records per launch.
    kern = kt["elementwise"]
    bracket_ms = kern["ms"] / max(kern["launches"], 1)
    avg_ms = ms_local / max(args.steps, 1)
    plan_lines = [ln.strip() for ln in ctx.dump_plan().splitlines()]
    compiled_as = next((ln[len("compiled: "):] for ln in plan_lines if ln.startswith("compiled: ")), "no")
    kernel_name = (f"lt_c_ew<{compiled_as}> (ahead-of-time compiled program)" if st["launches_compiled"] and compiled_as != "no"
                   else "lt_ew_kernel<fast> (interpreter)")
    achieved = nbytes / (avg_ms / 1e3) / 1e9 if avg_ms > 0 else 0.0
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": ncu_traffic(), "peak_source": peak_src, "kernel": kernel_name,
                "launch_us": 1e3 * avg_ms, "host_us_per_step": host_us_per_step,
                "paced_by": "gpu" if host_us_per_step < 1e3 * avg_ms else "host (the figure is not the kernel's rate)",
                "allocator_calls_in_timed_region": int(st["allocator_calls"]),
                "bytes_per_launch": nbytes, "frac_of_8TBs_nominal": achieved / 8000.0,
                "timing": "events around the timed region / launches (one launch per step, back to back)",
                "launch_us_bracketed": 1e3 * bracket_ms,
                "frac_bracketed": (nbytes / (bracket_ms / 1e3) / 1e9 / peak) if bracket_ms > 0 else None}

    extra = {}
    if not args.no_extra:
        extra = extra_measurements(ctx, lt, torch, timed, step, sets, nbytes)
        extra["host_ns_per_barrier"] = {k: st[k] / max(st["barriers"], 1) for k in st if k.startswith("ns_")}
        extra["cache"] = {"compiles": st["compiles"], "hits": st["cache_hits"], "barriers": st["barriers"],
                          "traces_matched": st["traces_matched"]}
        # the timed steps repeat one another, so their traces are only matched against the previous one (no canonical
        # form, no hash); the same 200 steps with that switched off show what a barrier costs when the graph is built,
        # canonicalised, hashed and looked up every time
        plain = lt.LazyContext(device=ctx.device)
        plain.set_option("trace_match", 0)
        psets = [tuple(plain.from_device_ptr(ctx.device_ptr(t), t.dtype, t.shape) for t in sets[k]) for k in range(len(sets))]
        keep = [None] * len(psets)
        for i in range(len(psets) + 2):
            keep[i % len(psets)] = traces.mlp_epilogue(plain, *psets[i % len(psets)], primitive_gelu=False)
            plain.barrier()
        plain.reset_stats()
        for i in range(200):
            keep[i % len(psets)] = traces.mlp_epilogue(plain, *psets[i % len(psets)], primitive_gelu=False)
            plain.barrier()
        torch.cuda.synchronize()
        pst = plain.stats()
        extra["host_ns_per_barrier_graph_built_every_step"] = {k: pst[k] / max(pst["barriers"], 1) for k in pst if k.startswith("ns_")}
        extra["cache_graph_built_every_step"] = {"compiles": pst["compiles"], "hits": pst["cache_hits"], "barriers": pst["barriers"]}
        del keep, psets
        plain.close()
        extra["c5_data_parallel_adam_step"] = dp_adam
        # the same program on the other two tiers, beside the headline: the interpreter serves a program that is not in
        # the build-time table until the run-time specialiser has built its kernel
        oc = extra.get("other_configs", {}).get("c2", {})
        if "interpreted_gbs" in oc:
            roofline["same_graph_on_the_interpreter"] = {"achieved": oc["interpreted_gbs"], "frac": oc["interpreted_gbs"] / peak}
        if "specialised_gbs" in oc:
            roofline["same_graph_specialised_at_run_time"] = {"achieved": oc["specialised_gbs"], "frac": oc["specialised_gbs"] / peak}
    cpu = cpu_baseline() if world == 1 and not args.no_cpu else None

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / max(args.steps, 1), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "trace": "convert x3, add, gelu_tanh, add, convert (7 ops, 1 fused kernel)",
                   "l2": f"{N_SETS} rotating buffer sets ({N_SETS * nbytes / 1e6:.0f} MB) larger than L2",
                   "per_gpu_batch": list(SHAPE), "parallelism": f"replicas x{world}, no collective"},
        "roofline": roofline,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": world * (2 * 2 * SHAPE[0] * SHAPE[1] + 2 * SHAPE[1]),
                "d2h_bytes_per_step": world * 2 * SHAPE[0] * SHAPE[1], "steps": e2e_steps,
                "ms_per_step": e2e_ms / e2e_steps},
        "gpu_launches": int(st["kernels_launched"]) * world,
        "clocks": clocks,
    }
    if cpu:
        line["cpu_baseline"] = cpu
    if extra:
        line["extra"] = extra
    print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def extra_measurements(ctx, lt, torch, timed, step, sets, nbytes) -> dict:
    """Context numbers: unfused baseline, primitive-op trace, and the other configurations."""
    from workloads import configs, traces

    out = {}
    n = 200
    # the same graph traced from primitive ops (16 ops) instead of the gelu_tanh op
    for i in range(len(sets) + 2):
        step(i, True)
    ms = timed(n, lambda i: step(i, True))
    out["c2_primitive_trace_gbs"] = nbytes * n / (ms / 1e3) / 1e9
    # unfused: one kernel per traced op (same library, fusion off)
    un = lt.LazyContext(device=ctx.device)
    un.set_option("fusion", 0)
    usets = [tuple(un.from_device_ptr(ctx.device_ptr(t), "bf16", t.shape) for t in s) for s in sets]
    keep = [None] * len(usets)

    def ustep(i, primitive=False):
        X, H, Bv = usets[i % len(usets)]
        keep[i % len(usets)] = traces.mlp_epilogue(un, X, H, Bv, primitive_gelu=primitive)
        un.barrier()

    for prim, key in ((False, "c2_unfused_gbs"), (True, "c2_primitive_unfused_gbs")):
        for i in range(len(usets) + 2):
            ustep(i, prim)
        ms = timed(50, lambda i: ustep(i, prim))
        out[key] = nbytes * 50 / (ms / 1e3) / 1e9
    un.set_kernel_timing(False)
    ms_f = timed(n, step)
    out["c2_fused_gbs"] = nbytes * n / (ms_f / 1e3) / 1e9
    # the same fused graph on the interpreter kernel (ahead-of-time compiled kernels switched off)
    ctx.set_option("compiled", 0)
    for i in range(len(sets) + 2):
        step(i)
    ms_i = timed(n, step)
    ctx.set_option("compiled", 1)
    out["c2_fused_interpreted_gbs"] = nbytes * n / (ms_i / 1e3) / 1e9
    out["c2_speedup_vs_unfused"] = out["c2_fused_gbs"] / out["c2_unfused_gbs"]
    out["c2_primitive_speedup_vs_unfused"] = out["c2_primitive_trace_gbs"] / out["c2_primitive_unfused_gbs"]
    keep.clear()
    del usets
    un.close()
    # replay: the same step without recording, canonicalising or hashing (one lt_replay call per step)
    X, H, Bv = sets[0]
    o = traces.mlp_epilogue(ctx, X, H, Bv, primitive_gelu=False)
    ctx.barrier()
    ms_r = timed(n, lambda i: ctx.replay())
    out["c2_replay_gbs"] = nbytes * n / (ms_r / 1e3) / 1e9
    del o
    out.update(adam_steps(lt, torch, ctx.device))
    out["other_configs"] = other_configs(lt, torch, ctx.device)
    out["wider_reductions"] = wider_reductions(lt, torch, ctx.device)
    return out


def data_parallel_adam(lt, torch, device: int, world: int, steps: int = 50) -> dict:
    """Second workload at any N: the synchronous data-parallel Adam step over the 161 ResNet-50 tensors -- the
    gradient buffer all-reduced over the ranks bucket by bucket (NCCL; nothing to exchange at N = 1), then the
    fused multi-tensor update, recorded once and replayed.  Device time per step, maximum over ranks."""
    from paper_2102_13267_b200.data_parallel import DataParallelAdam
    from workloads import configs
    from workloads.resnet50 import parameter_shapes

    ctx = lt.LazyContext(device=device)
    dp = DataParallelAdam(ctx, parameter_shapes())
    dp.flat["p"].normal_(0.0, 0.05)
    dp.flat["g"].normal_(0.0, 1e-3)
    for _ in range(3):
        dp.step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        dp.step()
    e1.record()
    torch.cuda.synchronize()
    ms = max_over_ranks(e0.elapsed_time(e1), world, torch.device("cuda", device)) / steps
    st = ctx.stats()
    nbytes = configs.algorithmic_bytes("c5")
    res = {"ms_per_step": ms, "adam_gbs_all_ranks": world * nbytes / ms / 1e6, "all_reduce_bytes_per_rank": 4 * dp.total,
           "buckets": len(dp.buckets), "compiles": st["compiles"], "replays": st["replays"], "world": world}
    ctx.close()
    return res


def other_configs(lt, torch, device: int) -> dict:
    """C1 to C4: fused, interpreted, specialised and unfused GB/s, flushes over rotating buffer sets (> 1 GB together) queued behind
    a busy stream and timed between two events (kernel time including the gap to the next launch)."""
    import math as _m

    from workloads import configs, traces

    dev = torch.device("cuda", device)
    peak, _ = measured_peak()

    def bf16(shape, std=1.0):
        return (torch.randn(shape, device=dev) * std).to(torch.bfloat16)

    def c1_make(c):
        return [c.from_torch(torch.rand(configs.FULL["c1"], device=dev) * 2 - 1) for _ in range(4)]

    def c3_make(c):
        sh = configs.FULL["c3"]
        return (c.from_torch(bf16(sh)), c.from_torch(bf16(sh)), c.from_torch(1 + 0.02 * torch.randn(sh[1], device=dev)),
                c.from_torch(0.02 * torch.randn(sh[1], device=dev)))

    def c4_make(c):
        return (c.from_torch(bf16(configs.FULL["c4"], 4.0)),)

    def c2_make(c):
        sh = configs.FULL["c2"]
        return (c.from_torch(bf16(sh)), c.from_torch(bf16(sh)), c.from_torch(bf16((sh[1],), 0.02)))

    cases = {
        "c1": (c1_make, lambda c, s: traces.elementwise_chain(c, *s)),
        "c2": (c2_make, lambda c, s: traces.mlp_epilogue(c, *s, primitive_gelu=False)),
        "c3": (c3_make, lambda c, s: traces.residual_dropout_layernorm(c, *s, shape=configs.FULL["c3"], p=0.1, eps=1e-5,
                                                                        seed=1, offset=0)),
        "c4": (c4_make, lambda c, s: traces.causal_softmax(c, *s, shape=configs.FULL["c4"], scale=1 / _m.sqrt(128))),
    }
    res = {}
    for name, (make, trace) in cases.items():
        nbytes = configs.algorithmic_bytes(name)
        nsets = max(2, _m.ceil(1.2e9 / nbytes))
        entry = {}
        # fused: the build-time kernel of the graph; interpreted: the same fused program on the interpreter kernels (what
        # a graph runs on until a kernel has been built for it); specialised: the kernel the run-time specialiser builds
        # for a program without a table entry (here: the table ignored); unfused: one kernel per traced op
        for mode, iters in (("fused", 40), ("interpreted", 20), ("specialised", 40), ("unfused", 10)):
            if name == "c2" and mode == "unfused":
                continue  # (measured above on the benchmark's own buffers)
            c = lt.LazyContext(device=device)
            if mode == "unfused":
                c.set_option("fusion", 0)
            elif mode == "interpreted":
                c.set_option("compiled", 0)
            elif mode == "specialised":
                c.set_option("debug.ignore_table", 1)
                c.set_option("specialise", 1)
            sets = [make(c) for _ in range(nsets)]
            keep = [None] * nsets
            warm = nsets + 2  # every set flushed once: no allocator call is left for the timed flushes
            for i in range(warm):
                keep[i % nsets] = trace(c, sets[i % nsets])
                c.barrier()
            torch.cuda.synchronize()
            c.reset_stats()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda._sleep(int(4e-3 * 1.9e9))  # the flushes queue up behind this and then run back to back
            e0.record()
            for i in range(iters):
                keep[i % nsets] = trace(c, sets[i % nsets])
                c.barrier()
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / iters
            entry[f"{mode}_us"] = 1e3 * ms
            entry[f"{mode}_gbs"] = nbytes / ms / 1e6
            entry[f"{mode}_launches"] = c.stats()["kernels_launched"] // iters
            entry[f"{mode}_allocator_calls"] = c.stats()["allocator_calls"]
            del keep, sets
            c.close()
        entry["frac_of_measured_peak"] = entry["fused_gbs"] / peak
        entry["interpreted_frac_of_measured_peak"] = entry["interpreted_gbs"] / peak
        entry["specialised_frac_of_measured_peak"] = entry["specialised_gbs"] / peak
        if "unfused_us" in entry:
            entry["speedup_vs_unfused"] = entry["unfused_us"] / entry["fused_us"]
        res[name] = entry
    return res


def wider_reductions(lt, torch, device: int) -> dict:
    """Beyond the five configurations: rows of 16384 columns (cluster row kernel) and reductions of computed values
    (first stage inside the computing kernel), each against the plan without that kernel.  Timed like other_configs."""
    import math as _m

    from workloads import idioms

    dev = torch.device("cuda", device)
    peak, _ = measured_peak()

    def inputs(c, kinds, shape):
        out = []
        for k in kinds:
            t = torch.randn(shape if k.startswith("mat") else (shape[-1],), device=dev)
            out.append(c.from_torch(t.to(torch.bfloat16) if k.endswith("bf16") else t))
        return out

    long_shape, red_shape = (8192, 16384), (16384, 4096)
    cases = []
    for name in ("softmax_bf16", "layernorm_bf16"):
        _, kinds, trace = next(e for e in idioms.ALL if e[0] == name)
        cases.append((f"{name}_16384_columns", kinds, trace, long_shape, 2 * 2 * long_shape[0] * long_shape[1], {"debug.cluster": 1}, "cta_per_row"))
    for name in ("sum_squares_f32", "relu_bias_grad_bf16"):
        _, kinds, trace = next(e for e in idioms.REDUCED if e[0] == name)
        nbytes = sum((2 if k.endswith("bf16") else 4) * red_shape[0] * red_shape[1] for k in kinds)
        cases.append((name, kinds, trace, red_shape, nbytes, {"specialise": 0, "debug.ignore_table": 1}, "unfused"))
    res = {}
    for name, kinds, trace, shape, nbytes, other, other_name in cases:
        entry = {}
        for mode, opts in (("", {}), (other_name, other)):
            c = lt.LazyContext(device=device)
            for k, v in opts.items():
                c.set_option(k, v)
            nsets = max(2, _m.ceil(1.2e9 / nbytes))
            sets = [inputs(c, kinds, shape) for _ in range(nsets)]
            keep = [None] * nsets
            for i in range(nsets + 2):
                keep[i % nsets] = trace(c, sets[i % nsets], shape[-1])
                c.barrier()
            torch.cuda.synchronize()
            iters = 20
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda._sleep(int(4e-3 * 1.9e9))
            e0.record()
            for i in range(iters):
                keep[i % nsets] = trace(c, sets[i % nsets], shape[-1])
                c.barrier()
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / iters
            pre = f"{mode}_" if mode else ""
            entry[f"{pre}us"] = 1e3 * ms
            entry[f"{pre}gbs"] = nbytes / ms / 1e6
            if not mode:
                entry["frac_of_measured_peak"] = entry["gbs"] / peak
            del keep, sets
            c.close()
        res[name] = entry
    return res


def adam_steps(lt, torch, device: int) -> dict:
    """C5: 100 Adam steps over the 161 ResNet-50 parameter tensors, one flush per step; traced every step
    (1 compile + 99 cache hits) against traced once and replayed 99 times.  Wall-clock per step, host included."""
    import math as _m

    from workloads import configs, traces
    from workloads.resnet50 import parameter_shapes

    shapes = parameter_shapes()
    nbytes = configs.algorithmic_bytes("c5")
    dev = torch.device("cuda", device)
    res = {}
    # the update of one parameter as one batched recording call (lt_op_many) instead of sixteen calls
    class _Refs:
        pass

    batch, refs = lt.Batch(), _Refs()
    b_in = [batch.input() for _ in range(4)]
    scalar_names = ("beta1", "one_minus_beta1", "beta2", "one_minus_beta2", "sqrt_bc2", "eps", "step_size")
    for name in scalar_names:
        setattr(refs, name, batch.input())
    traces.adam_update(batch, *b_in, refs)
    for mode in ("traced", "traced_batched", "replayed", "replayed_interpreted", "replayed_specialised"):
        ctx = lt.LazyContext(device=device)
        if mode == "replayed_interpreted":
            ctx.set_option("compiled", 0)
        elif mode == "replayed_specialised":
            ctx.set_option("debug.ignore_table", 1)
            ctx.set_option("specialise", 1)
        P, G, M, V = ([ctx.from_torch(torch.randn(s, device=dev) * 0.05) for s in shapes] for _ in range(4))
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        if mode == "traced":
            for step in range(1, 101):
                traces.adam_step(ctx, P, G, M, V, step=step)
                ctx.barrier()
        elif mode == "traced_batched":
            for step in range(1, 101):
                s = traces.AdamScalars(ctx, step=step)
                sc = [getattr(s, name) for name in scalar_names]
                for p, g, m, v in zip(P, G, M, V):
                    ctx.record(batch, [p, g, m, v, *sc])
                ctx.barrier()
        else:
            s = traces.AdamScalars(ctx, step=1)
            for p, g, m, v in zip(P, G, M, V):
                traces.adam_update(ctx, p, g, m, v, s)
            ctx.barrier()
            if mode == "replayed_specialised":  # the kernel was built while the graph was planned: not part of a step
                torch.cuda.synchronize()
                t0 = time.perf_counter()
            for step in range(2, 101):
                ctx.scalar_set(s.sqrt_bc2, _m.sqrt(1.0 - 0.999 ** step))
                ctx.scalar_set(s.step_size, 1e-3 / (1.0 - 0.9 ** step))
                ctx.replay()
        torch.cuda.synchronize()
        sec = time.perf_counter() - t0
        st = ctx.stats()
        res[f"c5_adam_100_steps_{mode}_ms_per_step"] = 10.0 * sec
        res[f"c5_adam_100_steps_{mode}_gbs"] = nbytes * 100 / sec / 1e9
        res[f"c5_adam_{mode}_cache"] = {"compiles": st["compiles"], "hits": st["cache_hits"], "replays": st["replays"],
                                         "kernels": st["kernels_launched"], "traces_matched": st["traces_matched"]}
        if mode == "traced_batched":
            res["c5_host_us_per_barrier_batched"] = {k: st[k] / 1e3 / max(st["barriers"], 1) for k in st if k.startswith("ns_")}
        if mode == "traced":
            res["c5_host_us_per_barrier"] = {k: st[k] / 1e3 / max(st["barriers"], 1) for k in st if k.startswith("ns_")}
        del P, G, M, V
        ctx.close()
    return res


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extra", action="store_true", help="skip the context measurements (unfused baseline etc.)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
