"""GPU parity of the wider reduction shapes against the CPU eager oracle: rows longer than a thread group keeps
in registers (fused long-row kernels and the split plan), column and whole-tensor reductions, outer broadcasts,
and the bounded device-side wait."""
import math

import numpy as np
import pytest

from helpers import assert_matches
from oracle.eager import EagerOracle, max_threads, set_threads
from workloads import configs, idioms, rng, traces

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lt():
    import paper_2102_13267_b200 as lt
    set_threads(max_threads())
    return lt


@pytest.fixture()
def ctx(lt):
    c = lt.LazyContext(device=0)
    yield c
    c.close()


def _idiom_inputs(kinds, shape, seed):
    g = rng.generator(seed, 9)
    arrs = []
    for k in kinds:
        what, dt = k.split(":")
        shp = shape if what == "mat" else (shape[-1],)
        a = rng.normal_f32(g, shp, 1.0, 1.0 if what == "vec" else 0.0)
        arrs.append((rng.to_bf16_bits(a) if dt == "bf16" else a, dt))
    return arrs


LONG_IDIOMS = ["softmax_bf16", "softmax_f32", "scaled_softmax_bf16", "layernorm_bf16", "layernorm_f32", "rmsnorm_bf16"]


@pytest.mark.parametrize("shape", [(5, 16384), (3, 65536), (4, 10000), (2, 8200), (300, 16384), (2, 3, 12288)])
@pytest.mark.parametrize("idiom", LONG_IDIOMS)
def test_listed_groups_on_long_rows_run_fused(ctx, idiom, shape):
    name, kinds, trace = next(e for e in idioms.ALL if e[0] == idiom)
    arrs = _idiom_inputs(kinds, shape, 61)
    O = EagerOracle()
    ref = trace(O, [O.leaf(a, d) for a, d in arrs], shape[-1])
    out = trace(ctx, [ctx.leaf(a, d) for a, d in arrs], shape[-1])
    ctx.barrier()
    st = ctx.stats()
    assert st["kernels_launched"] == 1 and st["launches_row"] == 1 and st["launches_compiled"] == 1, st
    assert_matches(ctx.fetch(out), ref.array, "f32" if name.endswith("f32") else "bf16", f"{name} {shape}")


# Rows of up to 65536 columns run with a thread-block cluster as the row's thread group; longer ones, and every long
# row when that kernel is switched off, are walked in slices by one CTA.  Both against the oracle, every cluster size,
# with the column vectors in registers / re-read and in shared memory, rows that do and do not fill the group.
@pytest.mark.parametrize("vectors", [0, 1])
@pytest.mark.parametrize("cluster", [1, 2, 4, 8])
@pytest.mark.parametrize("idiom,shape", [("layernorm_bf16", (9, 16384)), ("layernorm_f32", (5, 10000)), ("softmax_bf16", (7, 8200)),
                                         ("rmsnorm_bf16", (3, 32768)), ("layernorm_bf16", (3, 65536)), ("softmax_f32", (300, 12288)),
                                         # 4097 to 8192 columns with column vectors: two CTAs of a cluster instead of eight chunks per thread
                                         ("layernorm_bf16", (300, 8192)), ("layernorm_f32", (7, 6144)), ("rmsnorm_bf16", (5, 4104))])
def test_long_rows_in_every_cluster_shape(lt, idiom, shape, cluster, vectors):
    if cluster * 128 * 8 * 8 < shape[-1] and cluster != 1:
        pytest.skip("row too long for this cluster size")
    c = lt.LazyContext(device=0)
    c.set_option("debug.cluster", cluster)
    c.set_option("debug.cluster_vectors", vectors)
    name, kinds, trace = next(e for e in idioms.ALL if e[0] == idiom)
    arrs = _idiom_inputs(kinds, shape, 67)
    O = EagerOracle()
    ref = trace(O, [O.leaf(a, d) for a, d in arrs], shape[-1])
    out = trace(c, [c.leaf(a, d) for a, d in arrs], shape[-1])
    c.barrier()
    st = c.stats()
    assert st["kernels_launched"] == 1 and st["launches_row"] == 1 and st["launches_compiled"] == 1, st
    assert_matches(c.fetch(out), ref.array, "f32" if name.endswith("f32") else "bf16", f"{name} {shape} cluster {cluster} vectors {vectors}")
    c.close()


def test_rows_beyond_the_cluster_kernel_are_walked_in_slices(ctx):
    shape = (3, 131072)
    name, kinds, trace = next(e for e in idioms.ALL if e[0] == "softmax_bf16")
    arrs = _idiom_inputs(kinds, shape, 68)
    O = EagerOracle()
    ref = trace(O, [O.leaf(a, d) for a, d in arrs], shape[-1])
    out = trace(ctx, [ctx.leaf(a, d) for a, d in arrs], shape[-1])
    ctx.barrier()
    st = ctx.stats()
    assert st["kernels_launched"] == 1 and st["launches_compiled"] == 1, st
    assert_matches(ctx.fetch(out), ref.array, "bf16", "softmax 131072")


@pytest.mark.parametrize("depth", [0, 1, 2])
def test_long_row_staging_depths_agree(lt, depth):
    """Rows staged in shared memory two ahead, one ahead, or read from global memory in every pass."""
    shape = (37, 16384)
    c = lt.LazyContext(device=0)
    c.set_option("debug.compiled_depth", depth)
    x, h, g, b = configs.c3_inputs(62, shape)
    O = EagerOracle()
    kw = dict(shape=shape, p=0.1, eps=1e-5, seed=0xABCDEF, offset=3)
    zr, kr = traces.residual_dropout_layernorm(O, O.leaf(x, "bf16"), O.leaf(h, "bf16"), O.leaf(g, "f32"), O.leaf(b, "f32"), **kw)
    z, k = traces.residual_dropout_layernorm(c, c.leaf(x, "bf16"), c.leaf(h, "bf16"), c.leaf(g, "f32"), c.leaf(b, "f32"), **kw)
    c.barrier()
    st = c.stats()
    assert st["kernels_launched"] == 1 and st["launches_compiled"] == 1
    assert_matches(c.fetch(k), kr.array, "u8", "long c3 mask")
    assert_matches(c.fetch(z), zr.array, "bf16", "long c3 z")
    c.close()


def test_causal_softmax_on_long_rows(ctx):
    shape = (1, 20, 16384)
    s = configs.c4_inputs(63, shape)
    O = EagerOracle()
    ref = traces.causal_softmax(O, O.leaf(s, "bf16"), shape=shape, scale=1 / math.sqrt(128))
    y = traces.causal_softmax(ctx, ctx.leaf(s, "bf16"), shape=shape, scale=1 / math.sqrt(128))
    ctx.barrier()
    assert ctx.stats()["launches_compiled"] == 1
    got = ctx.fetch(y)
    assert_matches(got, ref.array, "bf16", "long causal softmax")
    assert (got[0, 3, 4:] == 0).all()


def test_in_place_softmax_on_long_rows(ctx):
    shape = (150, 16384)
    name, kinds, trace = next(e for e in idioms.ALL if e[0] == "softmax_bf16")
    arrs = _idiom_inputs(kinds, shape, 64)
    O = EagerOracle()
    ol, gl = [O.leaf(a, d) for a, d in arrs], [ctx.leaf(a, d) for a, d in arrs]
    ptr = ctx.device_ptr(gl[0])
    for _ in range(2):
        ol[0] = trace(O, ol, shape[-1])
        ctx.assign(gl[0], trace(ctx, gl, shape[-1]))
        ctx.barrier()
    st = ctx.stats()
    assert st["outputs_donated"] == 2 and st["outputs_allocated"] == 0 and ctx.device_ptr(gl[0]) == ptr
    assert_matches(ctx.fetch(gl[0]), ol[0].array, "bf16", "in-place long softmax")


def _unlisted(B, z):
    """A row-normalisation no kernel was instantiated for: |z - max| / (sum |z - max| + 3)."""
    d = B.op("abs", B.op("sub", z, B.op("row_max", z)))
    return B.op("div", d, B.op("add", B.op("row_sum", d), B.scalar(3.0)))


@pytest.mark.parametrize("shape", [(6, 16384), (3, 9001), (2, 70000), (40, 8193)])
def test_unlisted_long_row_graph_runs_split(ctx, shape):
    z = rng.normal_f32(rng.generator(65), shape, 1.0)
    O = EagerOracle()
    ref = _unlisted(O, O.leaf(z, "f32"))
    out = _unlisted(ctx, ctx.leaf(z, "f32"))
    ctx.barrier()
    st = ctx.stats()
    assert st["launches_reduce"] == 2 and st["launches_row"] == 0, st
    assert_matches(ctx.fetch(out), ref.array, "f32", f"split long rows {shape}")


def test_listed_group_with_unaligned_input_falls_back_to_the_split_plan(ctx):
    import torch

    shape = (7, 16384)
    name, kinds, trace = next(e for e in idioms.ALL if e[0] == "softmax_f32")
    (x, _), = _idiom_inputs(kinds, shape, 66)
    store = torch.zeros(x.size + 8, dtype=torch.float32, device="cuda:0")
    view = store[1:1 + x.size]  # 4-byte aligned only
    view.copy_(torch.from_numpy(x.reshape(-1)).to("cuda:0"))
    t = ctx.from_device_ptr(view.data_ptr(), "f32", shape, keep=store)
    O = EagerOracle()
    ref = trace(O, [O.leaf(x, "f32")], shape[-1])
    out = trace(ctx, [t], shape[-1])
    ctx.barrier()
    st = ctx.stats()
    assert st["launches_reduce"] == 2 and st["launches_row"] == 0, st
    assert "kernels of their own" in ctx.dump_plan()
    assert_matches(ctx.fetch(out), ref.array, "f32", "split fallback")
    # the same graph on an aligned input afterwards: the cached plan's fused kernel
    t2 = ctx.leaf(x, "f32")
    out2 = trace(ctx, [t2], shape[-1])
    ctx.barrier()
    st2 = ctx.stats()
    assert st2["cache_hits"] == 1 and st2["launches_row"] == 1
    assert_matches(ctx.fetch(out2), ref.array, "f32", "fused after fallback")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", [(1, 1), (3, 5), (1000, 7), (257, 96), (4, 3, 130), (5000,), (20000, 33), (64, 4096)])
def test_column_and_whole_tensor_reductions(ctx, dtype, shape):
    x = rng.normal_f32(rng.generator(67), shape, 2.0)
    a = x if dtype == "f32" else rng.to_bf16_bits(x)
    O = EagerOracle()
    ox, gx = O.leaf(a, dtype), ctx.leaf(a, dtype)
    names = ["col_sum", "col_max", "col_min", "all_sum", "all_max", "all_min"]
    outs = [ctx.op(n, gx) for n in names]
    ctx.barrier()
    assert ctx.stats()["launches_reduce"] == 6
    for n, t in zip(names, outs):
        ref = O.op(n, ox)
        assert_matches(ctx.fetch(t), ref.array, dtype, f"{n} {dtype} {shape}")


def test_reduction_results_feed_later_groups(ctx):
    shape = (300, 72)
    x = rng.normal_f32(rng.generator(68), shape, 1.0)
    O = EagerOracle()

    def graph(B, t):
        centred = B.op("sub", t, B.op("mul", B.op("col_sum", t), B.scalar(1.0 / shape[0])))      # column means removed
        scaled = B.op("div", centred, B.op("add", B.op("all_max", B.op("abs", centred)), B.scalar(1.0)))  # global scale
        return B.op("add", scaled, B.op("row_max", scaled))

    ref = graph(O, O.leaf(x, "f32"))
    out = graph(ctx, ctx.leaf(x, "f32"))
    ctx.barrier()
    assert ctx.stats()["launches_reduce"] == 2
    assert_matches(ctx.fetch(out), ref.array, "f32", "reductions feeding groups")


def test_outer_broadcast(ctx):
    g = rng.generator(69)
    r, cv = rng.normal_f32(g, (37, 1)), rng.normal_f32(g, (1, 100))
    O = EagerOracle()
    for name in ("mul", "sub", "max"):
        ref = O.op(name, O.leaf(r, "f32"), O.leaf(cv, "f32"))
        got = ctx.fetch(ctx.op(name, ctx.leaf(r, "f32"), ctx.leaf(cv, "f32")))
        assert_matches(got, ref.array, "f32", f"outer {name}", exact=True)
        ref = O.op(name, O.leaf(cv.reshape(100), "f32"), O.leaf(r, "f32"))
        got = ctx.fetch(ctx.op(name, ctx.leaf(cv.reshape(100), "f32"), ctx.leaf(r, "f32")))
        assert_matches(got, ref.array, "f32", f"outer {name} swapped", exact=True)


def test_bounded_wait_gives_up_and_is_reported(lt):
    """The kernel that stages long rows waits for its copies with a time limit.  Here the limit runs out on a wait
    nothing can satisfy (no copy is involved): the next blocking call reports it, and the context stays usable."""
    c = lt.LazyContext(device=0)
    x = c.leaf(np.arange(64, dtype=np.float32).reshape(8, 8), "f32")
    c.debug_wait_probe(2_000_000)  # 2 ms
    with pytest.raises(lt.LazyTensorError) as err:
        c.barrier(blocking=True)
    assert err.value.status == lt.STATUS_NAMES.index("LT_ERR_DEVICE_TIMEOUT")
    c.barrier(blocking=True)  # reported once
    np.testing.assert_array_equal(c.fetch(x + 1.0), np.arange(64, dtype=np.float32).reshape(8, 8) + 1)
    c.close()


def test_degenerate_and_mixed_cases(ctx):
    O = EagerOracle()
    g = rng.generator(90)
    # a single long row; a long row next to short work in the same flush
    x = rng.normal_f32(g, (1, 20000), 1.0)
    y = rng.normal_f32(g, (33, 64), 1.0)
    ox, gx, oy, gy = O.leaf(x, "f32"), ctx.leaf(x, "f32"), O.leaf(y, "f32"), ctx.leaf(y, "f32")
    outs_o = [O.op("row_sum", ox), O.op("sub", ox, O.op("row_max", ox)), O.op("exp", oy), O.op("all_min", oy)]
    outs_g = [ctx.op("row_sum", gx), ctx.op("sub", gx, ctx.op("row_max", gx)), ctx.op("exp", gy), ctx.op("all_min", gy)]
    ctx.barrier()
    for k, (r, t) in enumerate(zip(outs_o, outs_g)):
        assert_matches(ctx.fetch(t), r.array, "f32", f"mixed flush output {k}")
    # reductions of reductions, and a rank-0 result used twice
    m = ctx.op("all_max", ctx.op("col_sum", gy))
    mo = O.op("all_max", O.op("col_sum", oy))
    z = ctx.op("mul", ctx.op("sub", gy, m), m)
    zo = O.op("mul", O.op("sub", oy, mo), mo)
    assert_matches(ctx.fetch(z), zo.array, "f32", "rank-0 result used twice")
    assert_matches(ctx.fetch(m), mo.array, "f32", "rank-0 result fetched")


def test_replay_of_a_graph_with_reduction_kernels_and_a_view(lt):
    """lt_replay re-runs a plan that holds a column reduction (two stages through a plan temporary) and an in-place
    update through a narrow."""
    import torch

    c = lt.LazyContext(device=0)
    shape = (2000, 96)
    x0 = rng.normal_f32(rng.generator(91), shape, 1.0)
    xd = torch.from_numpy(x0).cuda()
    x = c.from_torch(xd)
    O = EagerOracle()
    ox = O.leaf(x0, "f32")

    def step(B, t):
        centred = B.op("sub", t, B.op("mul", B.op("col_sum", t), B.scalar(1.0 / shape[0])))
        v = B.view_narrow(t, 1, 32, 32)
        B.assign(t, B.op("mul", centred, B.scalar(0.5)))
        B.assign(v, B.op("add", v, B.scalar(1.0)))
        return v

    keep = step(c, x)
    c.barrier()
    ok = step(O, ox)
    for _ in range(3):
        c.replay()
        step(O, ox)
    st = c.stats()
    assert st["replays"] == 3 and st["compiles"] == 1
    assert_matches(c.fetch(x), ox.array, "f32", "base after three replays")
    assert_matches(c.fetch(keep), np.ascontiguousarray(ok.array), "f32", "view after three replays")
    c.close()


# ------------------------------------------------------------------ reductions fused with the computation of their input
def _sq_diff(B, a, b):
    d = B.op("sub", a, b)
    return B.op("mul", d, d)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", [(4096, 1024), (1000, 264), (33, 8), (5000, 40), (2, 3, 4096), (70000, 16)])
@pytest.mark.parametrize("name", ["col_sum", "col_max", "col_min", "all_sum", "all_max", "all_min"])
def test_reduction_of_a_computed_value_runs_inside_the_kernel_that_computes_it(lt, name, shape, dtype):
    """col / all reduction of an elementwise expression that nothing else reads: the expression's kernel reduces it
    (first stage) instead of storing it; the reduction group runs only its second stage."""
    c = lt.LazyContext(device=0)
    c.set_option("specialise", 1)  # the kernel for this (unlisted) program is built while the graph is planned
    g = rng.generator(71)
    a, b = rng.normal_f32(g, shape), rng.normal_f32(g, shape)
    if dtype == "bf16":
        a, b = rng.to_bf16_bits(a), rng.to_bf16_bits(b)
    O = EagerOracle()
    ref = O.op(name, _sq_diff(O, O.leaf(a, dtype), O.leaf(b, dtype)))
    out = c.op(name, _sq_diff(c, c.leaf(a, dtype), c.leaf(b, dtype)))
    c.barrier()
    plan, st = c.dump_plan(), c.stats()
    listed = "compiled: no" not in plan.split("launch 1:")[0]  # (a - b)^2 summed is one of the listed programs
    if "specialised at run time" not in plan and not listed:
        pytest.skip("the run-time compiler library is not installed")
    rows = int(np.prod(shape[:-1]))
    if rows >= 128 or (name.startswith("all") and rows * shape[-1] > 8192):  # large enough for two stages: fused
        assert "second stage only" in plan and "reduced-over-" in plan, plan
        assert st["kernels_launched"] == 2 and st["launches_specialised"] == (0 if listed else 1) and st["launches_compiled"] == 1, st
    assert_matches(c.fetch(out), ref.array, dtype, f"fused {name} {dtype} {shape}")
    c.close()


def test_fused_reduction_keeps_other_results_and_nan_semantics(lt):
    c = lt.LazyContext(device=0)
    c.set_option("specialise", 1)
    shape = (777, 512)
    x = rng.normal_f32(rng.generator(72), shape)
    x[5, 7] = np.nan
    O = EagerOracle()

    def graph(B, t):
        e = B.op("exp", B.op("mul", t, B.scalar(0.5)))          # also a result of its own
        m = B.op("col_max", B.op("abs", B.op("sub", e, t)))     # NaN in column 7 must come through
        return e, m

    (re, rm), (ge, gm) = graph(O, O.leaf(x, "f32")), graph(c, c.leaf(x, "f32"))
    c.barrier()
    if "specialised at run time" not in c.dump_plan():
        pytest.skip("the run-time compiler library is not installed")
    assert "second stage only" in c.dump_plan()
    assert_matches(c.fetch(ge), re.array, "f32", "value stored next to the reduction")
    got = c.fetch(gm)
    assert np.isnan(got[0, 7]) and np.isnan(rm.array[0, 7])
    assert_matches(got, rm.array, "f32", "column max with a NaN")
    c.close()


def test_fused_reduction_falls_back_when_it_cannot_run(lt):
    """Rows that are not whole chunks, a value that something else reads, and (default mode) the flushes before the
    specialiser has built the kernel all run the reduction on a materialised input -- same values."""
    O = EagerOracle()
    for shape, extra_reader in (((300, 100), False), ((512, 256), True)):
        c = lt.LazyContext(device=0)
        c.set_option("specialise", 1)
        a = rng.normal_f32(rng.generator(73), shape)
        oa, ga = O.leaf(a, "f32"), c.leaf(a, "f32")
        outs = []
        for B, t in ((O, oa), (c, ga)):
            sq = B.op("mul", t, t)
            r = B.op("col_sum", sq)
            outs.append((r, B.op("row_sum", sq) if extra_reader else None))
        c.barrier()
        assert "second stage only" not in c.dump_plan()
        assert_matches(c.fetch(outs[1][0]), outs[0][0].array, "f32", f"unfused {shape}")
        c.close()
    c = lt.LazyContext(device=0)  # default mode
    a = rng.normal_f32(rng.generator(74), (2048, 512))
    ref = O.op("all_sum", O.op("mul", O.leaf(a, "f32"), O.leaf(a, "f32"))).array
    ga = c.leaf(a, "f32")
    import time
    deadline, fused_flushes, flushes = time.time() + 90, 0, 0
    while time.time() < deadline and fused_flushes < 2:
        out = c.op("all_sum", c.op("mul", ga, ga))
        before = c.stats()["launches_specialised"]
        c.barrier()
        flushes += 1
        assert_matches(c.fetch(out), ref, "f32", f"flush {flushes}")
        fused_flushes += c.stats()["launches_specialised"] - before
        time.sleep(0.05)
    if "specialised at run time" in c.dump_plan():
        assert fused_flushes >= 2 and flushes >= 5, (flushes, c.stats())
    c.close()


@pytest.mark.parametrize("shape", [(2048, 1024), (777, 136), (40000, 8)])
@pytest.mark.parametrize("idiom", [e[0] for e in idioms.REDUCED])
def test_listed_reductions_of_computed_values(ctx, idiom, shape):
    """Gradient norms, squared errors, bias gradients, scales: kernels built ahead of time, fused from the first flush."""
    name, kinds, trace = next(e for e in idioms.REDUCED if e[0] == idiom)
    arrs = _idiom_inputs(kinds, shape, 75)
    O = EagerOracle()
    ref = trace(O, [O.leaf(a, d) for a, d in arrs], shape[-1])
    out = trace(ctx, [ctx.leaf(a, d) for a, d in arrs], shape[-1])
    ctx.barrier()
    plan, st = ctx.dump_plan(), ctx.stats()
    assert f"compiled: {name}" in plan and "second stage only" in plan, plan
    assert st["kernels_launched"] == 2 and st["launches_compiled"] == 1 and st["launches_specialised"] == 0, st
    assert_matches(ctx.fetch(out), ref.array, "f32", f"{name} {shape}")


@pytest.mark.parametrize("shape", [(3000, 512), (513, 72)])
def test_several_reductions_of_values_one_group_computes(lt, shape):
    """LayerNorm-backward style: column sums of dy * xhat and of dy, and a column maximum, from one pass over the inputs."""
    c = lt.LazyContext(device=0)
    c.set_option("specialise", 1)
    g = rng.generator(76)
    dy, xh = rng.to_bf16_bits(rng.normal_f32(g, shape)), rng.to_bf16_bits(rng.normal_f32(g, shape))
    O = EagerOracle()

    def graph(B, a, b):
        af, bf = B.op("convert", a, dtype="f32"), B.op("convert", b, dtype="f32")
        return [B.op("col_sum", B.op("mul", af, bf)), B.op("col_sum", B.op("mul", af, B.scalar(1.0))),
                B.op("col_max", B.op("abs", B.op("sub", af, bf)))]

    ref = graph(O, O.leaf(dy, "bf16"), O.leaf(xh, "bf16"))
    out = graph(c, c.leaf(dy, "bf16"), c.leaf(xh, "bf16"))
    c.barrier()
    plan, st = c.dump_plan(), c.stats()
    if "specialised at run time" not in plan:
        pytest.skip("the run-time compiler library is not installed")
    assert plan.count("second stage only") == 3 and plan.count("reduced-over-rows") == 3, plan
    assert st["kernels_launched"] == 4 and st["launches_specialised"] == 1, st
    for k, (t, r) in enumerate(zip(out, ref)):
        assert_matches(c.fetch(t), r.array, "f32", f"reduction {k} {shape}")
    c.close()
