"""lt_replay: running the previously flushed graph again without recording it (the paper's Section 8 proposal
to let users guarantee that a step's computation stays the same)."""
import math

import numpy as np
import pytest

import paper_2102_13267_b200 as lt
from helpers import assert_matches
from workloads import configs, traces
from workloads.resnet50 import parameter_shapes


def status(name):
    return lt.STATUS_NAMES.index(name)


# ------------------------------------------------------------------ host logic (no GPU)
@pytest.fixture()
def dry():
    c = lt.LazyContext(device=None)
    yield c
    c.close()


def fake(ctx, shape, dtype="f32", base=[1 << 32]):
    base[0] += 1 << 28
    return ctx.from_device_ptr(base[0], dtype, shape)


def test_replay_skips_recording_and_hashing(dry):
    a, b, c, d = (fake(dry, (64, 64)) for _ in range(4))
    y = traces.elementwise_chain(dry, a, b, c, d)
    dry.barrier()
    before = dry.stats()
    for _ in range(5):
        dry.replay()
    after = dry.stats()
    assert after["replays"] == 5 and after["kernels_launched"] - before["kernels_launched"] == 5
    for k in ("nodes_recorded", "barriers", "compiles", "cache_hits", "ns_canonicalise", "ns_hash_lookup"):
        assert after[k] == before[k], k
    assert dry.is_materialised(y)
    assert dry.replay_slots() == 1  # the scalar 0.5


def test_replay_refuses_what_it_cannot_guarantee(dry):
    with pytest.raises(lt.LazyTensorError) as e:
        dry.replay()
    assert e.value.status == status("LT_ERR_INVALID_ARG")
    a, b = fake(dry, (8, 8)), fake(dry, (8, 8))
    y = dry.op("add", a, b)
    dry.barrier()
    z = dry.op("mul", y, y)  # pending work
    with pytest.raises(lt.LazyTensorError) as e:
        dry.replay()
    assert e.value.status == status("LT_ERR_INVALID_ARG") and "pending" in str(e.value)
    dry.barrier()            # now the last graph is z = y * y
    dry.replay()
    dry.release(y)           # its input is gone
    with pytest.raises(lt.LazyTensorError) as e:
        dry.replay()
    assert e.value.status == status("LT_ERR_INVALID_ARG") and "released" in str(e.value)
    del z
    # an input no tensor names: nothing to read the next step's value from
    p, q = fake(dry, (8, 8)), fake(dry, (8, 8))
    w = dry.op("add", p, q)
    dry.release(q)
    dry.barrier()
    with pytest.raises(lt.LazyTensorError) as e:
        dry.replay()
    assert e.value.status == status("LT_ERR_UNSUPPORTED")
    del w


def test_scalar_set_rules(dry):
    a = fake(dry, (8, 8))
    one, half = dry.scalar(1.0), dry.scalar(0.5)
    with pytest.raises(lt.LazyTensorError):
        dry.scalar_set(one, 2.0)       # 1 is part of the graph, not a run-time value
    with pytest.raises(lt.LazyTensorError):
        dry.scalar_set(a, 2.0)         # not a scalar
    y = dry.op("mul", a, half)
    with pytest.raises(lt.LazyTensorError) as e:
        dry.scalar_set(half, 0.25)     # a pending op reads it
    assert "pending" in str(e.value)
    dry.barrier()
    dry.scalar_set(half, 0.25)
    dry.replay()
    assert dry.stats()["compiles"] == 1
    del y


def test_in_place_replay_keeps_buffers_and_guards_aliases(dry):
    shapes = [(64,), (128,)]
    P, G, M, V = ([fake(dry, s) for s in shapes] for _ in range(4))
    ptrs = [dry.device_ptr(t) for t in P + M + V]
    traces.adam_step(dry, P, G, M, V, step=1)
    dry.barrier()
    for _ in range(3):
        dry.replay()
    st = dry.stats()
    assert st["outputs_allocated"] == 0 and st["outputs_donated"] == 4 * 6
    assert [dry.device_ptr(t) for t in P + M + V] == ptrs
    assert dry.replay_slots() == 7


# ------------------------------------------------------------------ on the GPU
@pytest.fixture()
def ctx():
    c = lt.LazyContext(device=0)
    yield c
    c.close()


@pytest.mark.gpu
def test_adam_steps_replayed_match_steps_traced(ctx):
    """Step 1 is traced, steps 2..6 are replayed with the two step-dependent scalars set: same bits as
    tracing every step, and the oracle's values."""
    from oracle.eager import EagerOracle

    shapes = parameter_shapes()[:12] + [(1000,)]
    p, g, m, v = configs.c5_inputs(21, shapes)
    O = EagerOracle()
    op, og, om, ov = ([O.leaf(a, "f32") for a in arrs] for arrs in (p, g, m, v))
    rp, rg, rm, rv = ([ctx.leaf(a, "f32") for a in arrs] for arrs in (p, g, m, v))
    ref_ctx = lt.LazyContext(device=0)
    tp, tg, tm, tv = ([ref_ctx.leaf(a, "f32") for a in arrs] for arrs in (p, g, m, v))
    steps = 6
    s = traces.AdamScalars(ctx, step=1)
    for q, gr, mm, vv in zip(rp, rg, rm, rv):
        traces.adam_update(ctx, q, gr, mm, vv, s)
    ctx.barrier()
    traces.adam_step(O, op, og, om, ov, step=1)
    traces.adam_step(ref_ctx, tp, tg, tm, tv, step=1)
    ref_ctx.barrier()
    for step in range(2, steps + 1):
        bc1, bc2 = 1.0 - 0.9 ** step, 1.0 - 0.999 ** step
        ctx.scalar_set(s.sqrt_bc2, math.sqrt(bc2))
        ctx.scalar_set(s.step_size, 1e-3 / bc1)
        ctx.replay()
        traces.adam_step(O, op, og, om, ov, step=step)
        traces.adam_step(ref_ctx, tp, tg, tm, tv, step=step)
        ref_ctx.barrier()
    st = ctx.stats()
    assert (st["barriers"], st["compiles"], st["replays"]) == (1, 1, steps - 1)
    for i in range(len(shapes)):
        for a, t, o in ((rp[i], tp[i], op[i]), (rm[i], tm[i], om[i]), (rv[i], tv[i], ov[i])):
            got = ctx.fetch(a)
            assert np.array_equal(got, ref_ctx.fetch(t))
            assert_matches(got, o.array, "f32", f"adam replay tensor {i}")
    ref_ctx.close()


@pytest.mark.gpu
def test_replay_reads_current_inputs_and_rebinds_fresh_outputs(ctx):
    """A graph with a fresh (not in-place) result: after the caller changes an input buffer, a replay
    gives the result for the new contents, in the same result tensor."""
    import torch

    from oracle.eager import EagerOracle

    shape = (96, 256)
    x, h, b = configs.c2_inputs(22, shape)
    dev = [torch.from_numpy(a.view(np.int16)).cuda() for a in (x, h, b)]
    X, H, B = (ctx.from_torch(t, "bf16") for t in dev)
    out = traces.mlp_epilogue(ctx, X, H, B, primitive_gelu=False)
    ctx.barrier()
    first = ctx.fetch(out)
    x2, h2, _ = configs.c2_inputs(23, shape)
    dev[0].copy_(torch.from_numpy(x2.view(np.int16)))
    dev[1].copy_(torch.from_numpy(h2.view(np.int16)))
    ctx.replay()
    second = ctx.fetch(out)
    O = EagerOracle()
    r1 = traces.mlp_epilogue(O, O.leaf(x, "bf16"), O.leaf(h, "bf16"), O.leaf(b, "bf16"), primitive_gelu=False)
    r2 = traces.mlp_epilogue(O, O.leaf(x2, "bf16"), O.leaf(h2, "bf16"), O.leaf(b, "bf16"), primitive_gelu=False)
    assert_matches(first, r1.array, "bf16", "traced step")
    assert_matches(second, r2.array, "bf16", "replayed step")
    assert not np.array_equal(first, second)
    st = ctx.stats()
    assert (st["barriers"], st["replays"], st["kernels_launched"]) == (1, 1, 2)


@pytest.mark.gpu
def test_replay_with_new_dropout_offset(ctx):
    """The random-bits offset is a run-time slot: set by index between replays, the mask follows."""
    from oracle.eager import EagerOracle

    shape = (16, 256)
    x, h, g, b = configs.c3_inputs(24, shape)
    L = [ctx.leaf(a, d) for a, d in ((x, "bf16"), (h, "bf16"), (g, "f32"), (b, "f32"))]
    kw = dict(shape=shape, p=0.1, eps=1e-5, seed=77)
    z, k = traces.residual_dropout_layernorm(ctx, *L, offset=5, **kw)
    ctx.barrier()
    O = EagerOracle()
    ol = [O.leaf(a, d) for a, d in ((x, "bf16"), (h, "bf16"), (g, "f32"), (b, "f32"))]
    _, k5 = traces.residual_dropout_layernorm(O, *ol, offset=5, **kw)
    z9, k9 = traces.residual_dropout_layernorm(O, *ol, offset=9, **kw)
    assert_matches(ctx.fetch(k), k5.array, "u8", "mask, traced")
    # slots in canonical order: find the offset slot by its recorded neighbours (seed, offset are consecutive)
    n = ctx.replay_slots()
    assert n == 6
    ctx.replay_set_slot(1, 9, integer=True)  # slot 0 = seed, slot 1 = offset (the philox op is visited first)
    ctx.replay()
    assert_matches(ctx.fetch(k), k9.array, "u8", "mask, replayed with offset 9")
    assert_matches(ctx.fetch(z), z9.array, "bf16", "z, replayed with offset 9")
