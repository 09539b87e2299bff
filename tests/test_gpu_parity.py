"""GPU parity: the CUDA library against the CPU eager oracle, element by element, on the same
seeded inputs, through the C ABI (ctypes binding)."""
import math

import numpy as np
import pytest

from helpers import assert_matches
from oracle.eager import EagerOracle, set_threads, max_threads
from workloads import configs, rng, traces
from workloads.resnet50 import parameter_shapes

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lt():
    import paper_2102_13267_b200 as lt
    set_threads(max_threads())
    return lt


@pytest.fixture(params=["compiled", "interpreted"])
def ctx(lt, request):
    """Every case runs twice: with the ahead-of-time compiled kernels allowed (the default; launches whose
    extents or pointers rule out 128-bit accesses still fall to the interpreter) and on the interpreter alone."""
    c = lt.LazyContext(device=0)
    c.set_option("compiled", 1 if request.param == "compiled" else 0)
    c.compiled_allowed = request.param == "compiled"
    yield c
    c.close()


def both(ctx, arrays_dtypes):
    """Leaves for the oracle and for the library from the same arrays."""
    O = EagerOracle()
    return O, [O.leaf(a, d) for a, d in arrays_dtypes], [ctx.leaf(a, d) for a, d in arrays_dtypes]


# ------------------------------------------------------------------ C1
@pytest.mark.parametrize("shape", [(1, 1), (3, 5), (37, 19), (64, 64), (1000,), (2051,), (256, 257), (1024, 1024)])
def test_c1_chain(ctx, shape):
    ins = [(a, "f32") for a in configs.c1_inputs(1, shape)]
    O, ol, gl = both(ctx, ins)
    ref = traces.elementwise_chain(O, *ol)
    for it in range(10):
        y = traces.elementwise_chain(ctx, *gl)
        ctx.barrier()
        if it in (0, 9):
            assert_matches(ctx.fetch(y), ref.array, "f32", f"c1 {shape}", exact=True)
        del y
    s = ctx.stats()
    assert (s["compiles"], s["cache_hits"]) == (1, 9)
    assert s["kernels_launched"] == 10


# ------------------------------------------------------------------ C2
@pytest.mark.parametrize("shape", [(33, 40), (17, 36), (1, 8), (5, 7), (128, 4096), (8192, 4096)])
@pytest.mark.parametrize("primitive", [True, False])
def test_c2_mlp_epilogue(ctx, shape, primitive):
    x, h, b = configs.c2_inputs(2, shape)
    O, ol, gl = both(ctx, [(x, "bf16"), (h, "bf16"), (b, "bf16")])
    ref = traces.mlp_epilogue(O, *ol, primitive_gelu=primitive)
    out = traces.mlp_epilogue(ctx, *gl, primitive_gelu=primitive)
    ctx.barrier()
    assert ctx.stats()["kernels_launched"] == 1
    if shape[1] % 8 == 0 and shape[0] > 1:  # (a one-row input is not a broadcast: another program)
        assert ctx.stats()["launches_compiled"] == (1 if ctx.compiled_allowed else 0)
    assert_matches(ctx.fetch(out), ref.array, "bf16", f"c2 {shape}")


# ------------------------------------------------------------------ C3
@pytest.mark.parametrize("shape", [(32, 256), (5, 1024), (7, 48), (3, 1000), (2, 2048), (2, 4096), (3, 8192), (9, 8),
                                   (4, 3, 64), (16384, 1024)])
@pytest.mark.parametrize("out_dtype", ["bf16", "f32"])
def test_c3_residual_dropout_layernorm(ctx, shape, out_dtype):
    x, h, g, b = configs.c3_inputs(3, shape)
    O, ol, gl = both(ctx, [(x, "bf16"), (h, "bf16"), (g, "f32"), (b, "f32")])
    kw = dict(shape=shape, p=0.1, eps=1e-5, seed=0xDEADBEEF12345, offset=7, out_dtype=out_dtype)
    zr, kr = traces.residual_dropout_layernorm(O, *ol, **kw)
    z, k = traces.residual_dropout_layernorm(ctx, *gl, **kw)
    ctx.barrier()
    assert ctx.stats()["kernels_launched"] == 1
    if shape[-1] % 8 == 0:
        assert ctx.stats()["launches_compiled"] == (1 if ctx.compiled_allowed else 0)
    assert_matches(ctx.fetch(k), kr.array, "u8", f"c3 mask {shape}")
    assert_matches(ctx.fetch(z), zr.array, out_dtype, f"c3 z {shape}")
    # a new offset gives a new mask without a recompile
    kw["offset"] = 8
    z2, k2 = traces.residual_dropout_layernorm(ctx, *gl, **kw)
    _, kr2 = traces.residual_dropout_layernorm(O, *ol, **kw)
    assert_matches(ctx.fetch(k2), kr2.array, "u8", "c3 mask, second offset")
    s = ctx.stats()
    assert (s["compiles"], s["cache_hits"]) == (1, 1)


@pytest.mark.parametrize("shape", [(32, 256), (7, 48), (3, 1000), (5, 2048), (3, 8192), (2048, 1024)])
def test_residual_layernorm_without_dropout(ctx, shape):
    x, h, g, b = configs.c3_inputs(13, shape)
    O, ol, gl = both(ctx, [(x, "bf16"), (h, "bf16"), (g, "f32"), (b, "f32")])
    zr = traces.residual_layernorm(O, *ol, shape=shape, eps=1e-5)
    z = traces.residual_layernorm(ctx, *gl, shape=shape, eps=1e-5)
    ctx.barrier()
    st = ctx.stats()
    assert st["kernels_launched"] == 1 and st["launches_compiled"] == (1 if ctx.compiled_allowed else 0)
    assert_matches(ctx.fetch(z), zr.array, "bf16", f"layernorm {shape}")


# ------------------------------------------------------------------ C4
@pytest.mark.parametrize("shape", [(2, 64, 64), (1, 130, 130), (3, 24, 24), (1, 8, 8), (2, 1000, 1000), (1, 4, 2048),
                                   (16, 2048, 2048)])
@pytest.mark.parametrize("out_dtype", ["bf16", "f32"])
def test_c4_causal_softmax(ctx, shape, out_dtype):
    s = configs.c4_inputs(4, shape)
    O, ol, gl = both(ctx, [(s, "bf16")])
    kw = dict(shape=shape, scale=1.0 / math.sqrt(128.0), out_dtype=out_dtype)
    ref = traces.causal_softmax(O, *ol, **kw)
    y = traces.causal_softmax(ctx, *gl, **kw)
    ctx.barrier()
    assert ctx.stats()["kernels_launched"] == 1
    if shape[-1] % 8 == 0:
        assert ctx.stats()["launches_compiled"] == (1 if ctx.compiled_allowed else 0)
    got = ctx.fetch(y)
    assert_matches(got, ref.array, out_dtype, f"c4 {shape}")
    # masked entries are exactly +0
    q, k = shape[-2], shape[-1]
    iu = np.triu_indices(q, 1, k)
    assert (got[..., iu[0], iu[1]] == 0).all()


# ------------------------------------------------------------------ C5
def _adam_case(ctx, shapes, steps, check_every=1):
    params, grads, ms, vs = configs.c5_inputs(5, shapes)
    O = EagerOracle()
    op, og, om, ov = ([O.leaf(a, "f32") for a in arrs] for arrs in (params, grads, ms, vs))
    gp, gg, gm, gv = ([ctx.leaf(a, "f32") for a in arrs] for arrs in (params, grads, ms, vs))
    ptrs = [ctx.device_ptr(t) for t in gp + gm + gv]
    for step in range(1, steps + 1):
        traces.adam_step(O, op, og, om, ov, step=step)
        traces.adam_step(ctx, gp, gg, gm, gv, step=step)
        ctx.barrier()
        if step % check_every == 0 or step == steps:
            for i in range(len(shapes)):
                for name, a, b in (("p", gp[i], op[i]), ("m", gm[i], om[i]), ("v", gv[i], ov[i])):
                    assert_matches(ctx.fetch(a), b.array, "f32", f"c5 step {step} {name}[{i}] {shapes[i]}")
    # in-place: every parameter, m and v still lives in its original buffer (donation)
    assert [ctx.device_ptr(t) for t in gp + gm + gv] == ptrs
    s = ctx.stats()
    assert (s["compiles"], s["cache_hits"]) == (1, steps - 1)
    assert s["outputs_allocated"] == 0 and s["outputs_donated"] == 3 * len(shapes) * steps
    return s


def test_c5_adam_small(ctx):
    shapes = parameter_shapes()[:14] + [(1000,), (7,), (3, 5, 1, 1)]
    s = _adam_case(ctx, shapes, steps=4)
    assert s["kernels_launched"] == 4  # one multi-tensor launch per step


def test_c5_adam_100_steps(ctx):
    """The workload as specified: 100 steps, one barrier per step, 1 compile + 99 cache hits, on a reduced set of
    the parameter shapes (the oracle runs every step too).  Three tensors are compared after every step, all of them
    after the last."""
    shapes = parameter_shapes()[:14] + [(1000,), (7,), (3, 5, 1, 1)]
    params, grads, ms, vs = configs.c5_inputs(55, shapes)
    O = EagerOracle()
    op, og, om, ov = ([O.leaf(a, "f32") for a in arrs] for arrs in (params, grads, ms, vs))
    gp, gg, gm, gv = ([ctx.leaf(a, "f32") for a in arrs] for arrs in (params, grads, ms, vs))
    ptrs = [ctx.device_ptr(t) for t in gp + gm + gv]
    watch = (0, 7, len(shapes) - 2)
    for step in range(1, 101):
        traces.adam_step(O, op, og, om, ov, step=step)
        traces.adam_step(ctx, gp, gg, gm, gv, step=step)
        ctx.barrier()
        for i in (watch if step < 100 else range(len(shapes))):
            for name, a, b in (("p", gp[i], op[i]), ("m", gm[i], om[i]), ("v", gv[i], ov[i])):
                assert_matches(ctx.fetch(a), b.array, "f32", f"c5 step {step} {name}[{i}] {shapes[i]}")
    assert [ctx.device_ptr(t) for t in gp + gm + gv] == ptrs
    s = ctx.stats()
    assert (s["compiles"], s["cache_hits"]) == (1, 99)
    assert s["kernels_launched"] == 100 and s["launches_multi"] == 100
    assert s["outputs_allocated"] == 0 and s["outputs_donated"] == 3 * len(shapes) * 100


def test_c5_adam_full_shapes(ctx):
    s = _adam_case(ctx, parameter_shapes(), steps=3, check_every=3)
    assert s["kernels_launched"] == 3 and s["launches_multi"] == 3
    assert s["launches_compiled"] == (3 if ctx.compiled_allowed else 0)
    assert s["bytes_planned"] == 3 * 715_596_896


def test_data_parallel_adam_step_on_one_rank(ctx):
    """The data-parallel step with a world of one (no exchange): flat buffers, the averaging scalar folded into the
    graph, recorded once and replayed."""
    from paper_2102_13267_b200.data_parallel import DataParallelAdam

    shapes = parameter_shapes()[:12] + [(1000,), (8, 3)]
    params, grads, ms, vs = configs.c5_inputs(56, shapes)
    dp = DataParallelAdam(ctx, shapes)
    import torch
    for i in range(len(shapes)):
        dp.view("p", i).copy_(torch.from_numpy(params[i]))
        dp.view("g", i).copy_(torch.from_numpy(grads[i]))
    O = EagerOracle()
    op, og, om, ov = ([O.leaf(a, "f32") for a in arrs] for arrs in (params, grads, ms, vs))
    for step in range(1, 6):
        s = traces.AdamScalars(O, step=step)
        for p, g, m, v in zip(op, og, om, ov):
            traces.adam_update(O, p, O.op("mul", g, O.scalar(1.0)), m, v, s)
        dp.step()
    st = ctx.stats()
    assert (st["compiles"], st["replays"], st["launches_multi"]) == (1, 4, 5)
    assert st["launches_compiled"] == (5 if ctx.compiled_allowed else 0)
    torch.cuda.synchronize()
    for i in range(len(shapes)):
        for which, ref in (("p", op[i]), ("m", om[i]), ("v", ov[i])):
            assert_matches(dp.view(which, i).cpu().numpy(), ref.array, "f32", f"dp adam {which}[{i}]")


# ------------------------------------------------------------------ unfused baseline
def test_unfused_matches_oracle(ctx):
    ctx.set_option("fusion", 0)
    shape = (6, 136)
    x, h, g, b = configs.c3_inputs(6, shape)
    O, ol, gl = both(ctx, [(x, "bf16"), (h, "bf16"), (g, "f32"), (b, "f32")])
    kw = dict(shape=shape, p=0.1, eps=1e-5, seed=3, offset=1)
    zr, kr = traces.residual_dropout_layernorm(O, *ol, **kw)
    z, k = traces.residual_dropout_layernorm(ctx, *gl, **kw)
    ctx.barrier()
    assert ctx.stats()["kernels_launched"] >= 15  # one kernel per traced op
    assert_matches(ctx.fetch(k), kr.array, "u8", "unfused mask")
    assert_matches(ctx.fetch(z), zr.array, "bf16", "unfused z")
    s = configs.c4_inputs(6, (2, 40, 40))
    O, ol, gl = both(ctx, [(s, "bf16")])
    ref = traces.causal_softmax(O, *ol, shape=(2, 40, 40), scale=0.1)
    y = traces.causal_softmax(ctx, *gl, shape=(2, 40, 40), scale=0.1)
    assert_matches(ctx.fetch(y), ref.array, "bf16", "unfused softmax")


# ------------------------------------------------------------------ common fusion groups (workloads/idioms.py)
def _idiom_inputs(kinds, shape, seed):
    g = rng.generator(seed, 9)
    arrs = []
    for k in kinds:
        what, dt = k.split(":")
        shp = shape if what == "mat" else (shape[-1],)
        a = rng.normal_f32(g, shp, 1.0, 1.0 if what == "vec" else 0.0)
        arrs.append((rng.to_bf16_bits(a) if dt == "bf16" else a, dt))
    return arrs


@pytest.mark.parametrize("shape", [(24, 64), (7, 1000), (5, 2048), (3, 40), (300, 1024)])
@pytest.mark.parametrize("idiom", [e[0] for e in __import__("workloads.idioms", fromlist=["ALL"]).ALL])
def test_common_fusion_groups(ctx, idiom, shape):
    from workloads import idioms

    name, kinds, trace = next(e for e in idioms.ALL if e[0] == idiom)
    O, ol, gl = both(ctx, _idiom_inputs(kinds, shape, 31))
    ref = trace(O, ol, shape[-1])
    out = trace(ctx, gl, shape[-1])
    ctx.barrier()
    st = ctx.stats()
    assert st["kernels_launched"] == 1 and st["launches_compiled"] == (1 if ctx.compiled_allowed else 0)
    dt = "f32" if name.endswith("f32") else "bf16"
    assert_matches(ctx.fetch(out), ref.array, dt, f"{name} {shape}")


def test_sgd_momentum_many_tensors(ctx):
    from workloads import idioms

    shapes = parameter_shapes()[:10] + [(1000,)]
    g = rng.generator(32, 9)
    host = [[rng.normal_f32(g, s, 0.1) for s in shapes] for _ in range(3)]
    O = EagerOracle()
    op, og, ob = ([O.leaf(a, "f32") for a in arrs] for arrs in host)
    gp, gg, gb = ([ctx.leaf(a, "f32") for a in arrs] for arrs in host)
    for _ in range(3):
        idioms.sgd_momentum(O, op, og, ob)
        idioms.sgd_momentum(ctx, gp, gg, gb)
        ctx.barrier()
    st = ctx.stats()
    assert st["kernels_launched"] == 3 and st["launches_multi"] == 3
    assert st["launches_compiled"] == (3 if ctx.compiled_allowed else 0)
    for a, r in zip(gp + gb, op + ob):
        assert_matches(ctx.fetch(a), r.array, "f32", "sgd momentum", exact=True)


@pytest.mark.parametrize("idiom", ["softmax_bf16", "residual_add_bf16"])
def test_in_place_update_through_a_compiled_kernel(ctx, idiom):
    """x := f(x, ...) with the result donated to x's buffer: the row kernel's staging ring reads blocks of rows
    ahead of the block being written, the elementwise kernel requests its inputs before it stores."""
    from workloads import idioms

    shape = (3000, 1024)  # more blocks of rows than resident CTAs, a ragged last wave
    name, kinds, trace = next(e for e in idioms.ALL if e[0] == idiom)
    O, ol, gl = both(ctx, _idiom_inputs(kinds, shape, 35))
    ptr = ctx.device_ptr(gl[0])
    for _ in range(2):
        O_out = trace(O, ol, shape[-1])
        ol[0] = O_out
        ctx.assign(gl[0], trace(ctx, gl, shape[-1]))
        ctx.barrier()
    st = ctx.stats()
    assert st["outputs_donated"] == 2 and st["outputs_allocated"] == 0 and ctx.device_ptr(gl[0]) == ptr
    assert st["launches_compiled"] == (2 if ctx.compiled_allowed else 0)
    assert_matches(ctx.fetch(gl[0]), ol[0].array, "bf16", f"in-place {name}")
