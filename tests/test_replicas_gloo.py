"""The N > 1 path is independent replicas: every rank traces and plans the same graph on its own buffers,
and the job time is the maximum over ranks.  Two gloo ranks on CPU with record-and-plan-only contexts."""
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
    import bench
    import paper_2102_13267_b200 as lt
    from workloads import configs, traces

    ctx = lt.LazyContext(device=None)
    leaves = [ctx.from_device_ptr((1 << 30) + (rank * 8 + i) * (1 << 26), "bf16", s)
              for i, s in enumerate([(64, 256), (64, 256), (256,)])]
    for _ in range(5):
        y = traces.mlp_epilogue(ctx, *leaves, primitive_gelu=False)
        ctx.barrier()
    st = ctx.stats()
    ms = bench.max_over_ranks(10.0 * (rank + 1), world)          # rank 1 is the slow one
    counts = torch.tensor([st["compiles"], st["cache_hits"], st["kernels_launched"]], dtype=torch.int64)
    gathered = [torch.zeros_like(counts) for _ in range(world)]
    dist.all_gather(gathered, counts)
    if rank == 0:
        out.put((ms, [g.tolist() for g in gathered], bench.aggregate_gbs(configs.algorithmic_bytes("c2", (64, 256)), 5, world, ms)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_over_gloo():
    world = 2
    ctxmp = mp.get_context("spawn")
    out = ctxmp.Queue()
    port = _free_port()
    procs = [ctxmp.Process(target=_rank, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    ms, counts, gbs = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ms == 20.0                                   # the maximum over ranks, not rank 0's own 10 ms
    assert counts == [[1, 4, 5], [1, 4, 5]]             # each replica: one compile, four hits, no exchange
    nbytes = 6 * 64 * 256 + 2 * 256
    assert abs(gbs - 2 * nbytes * 5 / 0.020 / 1e9) < 1e-12
