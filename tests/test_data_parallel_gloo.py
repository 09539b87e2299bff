"""The data-parallel Adam step with two gloo ranks on CPU: record-and-plan-only contexts (nothing is computed on
a device), gradient buffers reduced on CPU tensors.  Checks the host-side logic: bucket layout in launch order,
identical graphs and plans on every rank, summed gradients, one compile and replays afterwards."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank(rank: int, world: int, port: int, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import paper_2102_13267_b200 as lt
    from paper_2102_13267_b200.data_parallel import DataParallelAdam
    from workloads.resnet50 import parameter_shapes

    shapes = parameter_shapes()[:20] + [(1000,), (7,)]
    ctx = lt.LazyContext(device=None)
    dp = DataParallelAdam(ctx, shapes, bucket_bytes=64 << 10)
    for i in range(len(shapes)):
        dp.view("g", i).fill_(float(rank + 1) * (i + 1))
    for _ in range(4):
        dp.step()
    # buckets tile the flat buffer in order, every tensor inside exactly one
    assert dp.buckets[0][0] == 0 and dp.buckets[-1][1] == dp.total
    assert all(a[1] == b[0] for a, b in zip(dp.buckets, dp.buckets[1:])) and len(dp.buckets) > 2
    for off, n in zip(dp.offsets, dp.sizes):
        assert sum(lo <= off and off + n <= hi for lo, hi in dp.buckets) == 1 and off % 64 == 0
    st = ctx.stats()
    plan = ctx.dump_plan()
    # four all-reduces of a buffer nobody rewrites: (1 + 2) * 3^3 times tensor i's rank-independent factor
    sums = [float(dp.view("g", i).flatten()[0]) / (i + 1) for i in (0, 5, len(shapes) - 1)]
    info = (st["compiles"], st["cache_hits"], st["replays"], st["launches_multi"], plan, sums)
    gathered = [None] * world
    dist.all_gather_object(gathered, info)
    if rank == 0:
        out.put(gathered)
    dist.barrier()
    dist.destroy_process_group()


def test_data_parallel_adam_two_gloo_ranks():
    world = 2
    ctxmp = mp.get_context("spawn")
    out = ctxmp.Queue()
    port = _free_port()
    procs = [ctxmp.Process(target=_rank, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    gathered = out.get(timeout=180)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    a, b = gathered
    assert a[:4] == b[:4] == (1, 0, 3, 4)          # one graph planned, replayed three times, one launch per step
    assert a[4] == b[4]                            # the same plan text on both ranks (same program, same donation)
    assert "multi" in a[4] and a[4].count("launch ") == 1
    # rank 0's gradients after the reductions: start (1 + 2) -> x2 -> x2 -> x2 is wrong; each all-reduce sums the two
    # ranks' current buffers, which are equal after the first: 3, 6, 12, 24
    assert a[5] == b[5] == [24.0, 24.0, 24.0]
