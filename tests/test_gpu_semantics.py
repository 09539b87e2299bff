"""GPU semantics beyond the five configurations: every traced op against the oracle, in-place
hazards of the paper's Section 4.3, and randomly generated graphs (fused and unfused)."""
import numpy as np
import pytest

from helpers import assert_matches
from oracle.eager import EagerOracle
from workloads import rng

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lt():
    import paper_2102_13267_b200 as lt
    return lt


@pytest.fixture()
def ctx(lt):
    c = lt.LazyContext(device=0)
    yield c
    c.close()


def both(ctx, O, arr, dtype):
    return O.leaf(arr, dtype), ctx.leaf(arr, dtype)


FLOAT_UNARY = ["neg", "abs", "relu", "exp", "log", "tanh", "sqrt", "rsqrt", "recip", "square", "sigmoid", "gelu_tanh"]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", [(5, 24), (3, 7), (1000,)])
def test_float_unary_ops(ctx, dtype, shape):
    g = rng.generator(21)
    x = rng.normal_f32(g, shape, 2.0)
    pos = np.abs(x) + np.float32(0.05)
    for name in FLOAT_UNARY:
        arg = pos if name in ("log", "sqrt", "rsqrt", "recip") else x
        a = arg if dtype == "f32" else rng.to_bf16_bits(arg)
        O = EagerOracle()
        ol, gl = both(ctx, O, a, dtype)
        ref = O.op(name, ol)
        got = ctx.fetch(ctx.op(name, gl))
        assert_matches(got, ref.array, dtype, f"{name} {dtype} {shape}")


@pytest.mark.parametrize("other_shape", [None, (), (40,), (1, 40), (6, 1)])
def test_float_binary_ops_and_broadcast_classes(ctx, other_shape):
    g = rng.generator(22)
    shape = (6, 40)
    x = rng.normal_f32(g, shape, 2.0)
    y = rng.normal_f32(g, shape if other_shape is None else other_shape, 2.0)
    y = np.where(np.abs(y) < 0.1, np.float32(0.5), y).astype(np.float32)
    for name in ("add", "sub", "mul", "div", "max", "min", "gt", "ge", "lt", "le", "eq", "ne"):
        for swap in (False, True):
            O = EagerOracle()
            ox, gx = both(ctx, O, x, "f32")
            oy, gy = both(ctx, O, y, "f32")
            ref = O.op(name, *((oy, ox) if swap else (ox, oy)))
            out = ctx.op(name, *((gy, gx) if swap else (gx, gy)))
            assert_matches(ctx.fetch(out), ref.array, ref.dtype, f"{name} swap={swap} {other_shape}")
    # scalar operands on either side
    for name in ("sub", "div", "max", "lt"):
        for swap in (False, True):
            O = EagerOracle()
            ox, gx = both(ctx, O, x, "f32")
            args_o = (O.scalar(1.75), ox) if swap else (ox, O.scalar(1.75))
            args_g = (ctx.scalar(1.75), gx) if swap else (gx, ctx.scalar(1.75))
            ref = O.op(name, *args_o)
            assert_matches(ctx.fetch(ctx.op(name, *args_g)), ref.array, ref.dtype, f"{name} scalar swap={swap}")


def test_integer_mask_and_convert_ops(ctx):
    g = rng.generator(23)
    a = g.integers(-1000, 1000, size=(9, 16), dtype=np.int32)
    b = g.integers(-1000, 1000, size=(9, 16), dtype=np.int32)
    a[0, :4] = [2**31 - 1, -2**31, 0, -1]
    for dt, conv in (("i32", lambda v: v), ("u32", lambda v: v.view(np.uint32))):
        for name in ("add", "sub", "mul", "max", "min", "and", "or", "xor", "gt", "le", "eq", "ne"):
            O = EagerOracle()
            oa, ga = both(ctx, O, conv(a), dt)
            ob, gb = both(ctx, O, conv(b), dt)
            ref = O.op(name, oa, ob)
            assert_matches(ctx.fetch(ctx.op(name, ga, gb)), ref.array, ref.dtype, f"{name} {dt}")
    O = EagerOracle()
    oa, ga = both(ctx, O, a, "i32")
    for name in ("neg", "abs"):
        assert_matches(ctx.fetch(ctx.op(name, ga)), O.op(name, oa).array, "i32", name)
    m1 = (g.random((9, 16)) < 0.5).astype(np.uint8)
    m2 = (g.random((9, 16)) < 0.5).astype(np.uint8)
    om1, gm1 = both(ctx, O, m1, "u8")
    om2, gm2 = both(ctx, O, m2, "u8")
    for name in ("and", "or", "xor"):
        assert_matches(ctx.fetch(ctx.op(name, gm1, gm2)), O.op(name, om1, om2).array, "u8", name)
    assert_matches(ctx.fetch(ctx.op("not", gm1)), O.op("not", om1).array, "u8", "not")
    x = rng.normal_f32(g, (9, 16), 50.0)
    x[0, :5] = [np.nan, 3e9, -3e9, -0.0, 0.5]
    ox, gx = both(ctx, O, x, "f32")
    assert_matches(ctx.fetch(ctx.op("where", gm1, gx, ctx.scalar(0.0))), O.op("where", om1, ox, O.scalar(0.0)).array, "f32", "where")
    assert_matches(ctx.fetch(ctx.op("where", gm1, ctx.scalar(-np.inf), gx)), O.op("where", om1, O.scalar(-np.inf), ox).array, "f32", "where")
    for src, arr, dsts in (("f32", x, ("bf16", "i32", "u8")), ("i32", a, ("f32", "u32", "u8")), ("u8", m1 * 200, ("f32", "i32", "u32")),
                           ("u32", a.view(np.uint32), ("f32", "i32"))):
        o, gq = both(ctx, O, arr.astype({"f32": np.float32, "i32": np.int32, "u8": np.uint8, "u32": np.uint32}[src]), src)
        for dst in dsts:
            ref = O.op("convert", o, dtype=dst)
            assert_matches(ctx.fetch(ctx.op("convert", gq, dtype=dst)), ref.array, dst, f"convert {src}->{dst}")


def test_iota_philox_and_reductions(ctx):
    O = EagerOracle()
    for shape in [(7,), (5, 24), (2, 3, 16), (3, 10)]:
        for dim in range(len(shape)):
            ref = O.op("iota", shape=shape, dim=dim)
            assert_matches(ctx.fetch(ctx.op("iota", shape=shape, dim=dim)), ref.array, "i32", f"iota {shape} {dim}")
        ref = O.op("philox_bits", shape=shape, seed=2**63 + 5, offset=2**40 + 3)
        got = ctx.fetch(ctx.op("philox_bits", shape=shape, seed=2**63 + 5, offset=2**40 + 3))
        assert_matches(got, ref.array, "u32", f"philox {shape}")
    g = rng.generator(24)
    for shape in [(4, 8), (3, 40), (2, 3, 100), (5, 1), (2, 2048)]:
        x = rng.normal_f32(g, shape, 3.0)
        ox, gx = both(ctx, O, x, "f32")
        for name in ("row_sum", "row_max", "row_min"):
            assert_matches(ctx.fetch(ctx.op(name, gx)), O.op(name, ox).array, "f32", f"{name} {shape}")


# ------------------------------------------------------------------ paper Section 4.3 hazards
def test_in_place_twice_observed(ctx):
    a0 = np.arange(32, dtype=np.float32).reshape(4, 8)
    a = ctx.leaf(a0, "f32")
    a += 1.0
    first = ctx.fetch(a)
    second = ctx.fetch(a)          # must not increment again
    np.testing.assert_array_equal(first, a0 + 1)
    np.testing.assert_array_equal(second, a0 + 1)
    assert ctx.stats()["kernels_launched"] == 1 and ctx.stats()["outputs_donated"] == 1


def test_reader_of_old_value_survives_in_place_update(ctx):
    a0 = np.arange(64, dtype=np.float32).reshape(8, 8)
    for fusion in (1, 0):
        c = type(ctx)(device=0)
        c.set_option("fusion", fusion)
        a = c.leaf(a0, "f32")
        b = a + 2.0
        a += 1.0
        np.testing.assert_array_equal(c.fetch(a), a0 + 1)
        np.testing.assert_array_equal(c.fetch(b), a0 + 2)   # b saw the old a
        c.close()


def test_scalar_values_are_runtime_parameters(ctx):
    x0 = np.linspace(-2, 2, 96, dtype=np.float32).reshape(4, 24)
    x = ctx.leaf(x0, "f32")
    for k in (0.0, 1.0, 2.5, -7.0):
        np.testing.assert_array_equal(ctx.fetch(ctx.op("add", ctx.op("mul", x, ctx.scalar(k)), ctx.scalar(k))), x0 * np.float32(k) + np.float32(k))
    s = ctx.stats()
    assert s["compiles"] == 3 and s["cache_hits"] == 1  # graphs for 0, for 1, and one shared by 2.5 and -7


def test_ieee_option_is_bit_exact_for_adam(lt):
    from workloads import configs, traces
    c = lt.LazyContext(device=0)
    c.set_option("ieee", 1)
    shapes = [(64, 3, 7, 7), (64,), (1000,), (33,)]
    params, grads, ms, vs = configs.c5_inputs(9, shapes)
    O = EagerOracle()
    op, og, om, ov = ([O.leaf(a, "f32") for a in arrs] for arrs in (params, grads, ms, vs))
    gp, gg, gm, gv = ([c.leaf(a, "f32") for a in arrs] for arrs in (params, grads, ms, vs))
    for step in range(1, 4):
        traces.adam_step(O, op, og, om, ov, step=step)
        traces.adam_step(c, gp, gg, gm, gv, step=step)
    for a, r in zip(gp + gm + gv, op + om + ov):
        assert_matches(c.fetch(a), r.array, "f32", "adam ieee", exact=True)
    c.close()


# ------------------------------------------------------------------ random graphs
def _random_graph(B, g, leaves, n_ops):
    """Issues the same random op sequence on backend B; returns the values that stay live."""
    vals = list(leaves)
    for _ in range(n_ops):
        kind = g.integers(0, 10)
        full = [v for v in vals if v.shape == leaves[0].shape]
        x = full[g.integers(0, len(full))]
        if kind < 4:
            y = vals[g.integers(0, len(vals))]
            name = ["add", "sub", "mul", "max"][g.integers(0, 4)]
            vals.append(B.op(name, x, y) if g.integers(0, 2) else B.op(name, y, x))
        elif kind < 6:
            vals.append(B.op(["add", "mul", "sub"][g.integers(0, 3)], x, B.scalar(float(g.integers(-3, 4)) / 2)))
        elif kind < 8:
            vals.append(B.op(["tanh", "relu", "abs", "neg", "sigmoid", "square"][g.integers(0, 6)], x))
        elif kind == 8:
            vals.append(B.op(["row_sum", "row_max"][g.integers(0, 2)], x))
        else:
            m = B.op("gt", x, B.scalar(0.0))
            vals.append(B.op("where", m, x, full[g.integers(0, len(full))]))
    n_keep = int(g.integers(1, 4))
    return vals[-n_keep:]


@pytest.mark.parametrize("seed", range(12))
@pytest.mark.parametrize("fusion", [1, 0])
def test_random_graphs(lt, seed, fusion):
    shape = [(6, 40), (3, 17), (2, 4, 64), (5, 256)][seed % 4]
    gi = rng.generator(100 + seed)
    arrays = [rng.normal_f32(gi, shape, 1.0) for _ in range(3)] + [rng.normal_f32(gi, (shape[-1],), 1.0)]
    c = lt.LazyContext(device=0)
    c.set_option("fusion", fusion)
    O = EagerOracle()
    ref = _random_graph(O, rng.generator(500 + seed), [O.leaf(a, "f32") for a in arrays], 14)
    got = _random_graph(c, rng.generator(500 + seed), [c.leaf(a, "f32") for a in arrays], 14)
    c.barrier()
    for k, (r, t) in enumerate(zip(ref, got)):
        # long random chains amplify rounding differences of tanh/sigmoid: compare with a wider absolute term
        a, b = c.fetch(t), r.array
        assert a.shape == b.shape
        np.testing.assert_allclose(a, b, rtol=2e-4, atol=2e-4, equal_nan=True, err_msg=f"seed {seed} output {k}")
    c.close()


# ------------------------------------------------------------------ pointers that cannot take 128-bit accesses
@pytest.mark.parametrize("dtype,offset", [("f32", 1), ("f32", 2), ("bf16", 1), ("bf16", 3), ("u8", 5)])
def test_unaligned_device_pointers(ctx, dtype, offset):
    import torch
    from workloads import rng as R
    g = R.generator(31)
    shape = (37, 64)
    n = shape[0] * shape[1]
    tdt = {"f32": torch.float32, "bf16": torch.int16, "u8": torch.uint8}[dtype]

    def make(values_f32):
        if dtype == "f32":
            host = values_f32
        elif dtype == "bf16":
            host = R.to_bf16_bits(values_f32)
        else:
            host = (values_f32 > 0).astype(np.uint8)
        store = torch.zeros(n + 16, dtype=tdt, device="cuda:0")
        view = store[offset:offset + n]
        src = torch.from_numpy(host.view(np.int16) if dtype == "bf16" else host).reshape(-1).to("cuda:0")
        view.copy_(src)
        return host, ctx.from_device_ptr(view.data_ptr(), dtype, shape, keep=store)

    a_host, a = make(R.normal_f32(g, shape))
    b_host, b = make(R.normal_f32(g, shape))
    O = EagerOracle()
    oa, ob = O.leaf(a_host, dtype), O.leaf(b_host, dtype)
    if dtype == "u8":
        ref = O.op("xor", O.op("and", oa, ob), O.op("not", oa))
        got = ctx.op("xor", ctx.op("and", a, b), ctx.op("not", a))
    else:
        ref = O.op("sub", O.op("mul", oa, ob), O.op("relu", oa))
        got = ctx.op("sub", ctx.op("mul", a, b), ctx.op("relu", a))
    assert_matches(ctx.fetch(got), ref.array, dtype, f"unaligned {dtype}+{offset}")


def test_unaligned_instance_in_a_multi_tensor_launch(lt):
    import torch
    from workloads import configs, traces
    c = lt.LazyContext(device=0)
    shapes = [(96,), (40, 8), (1000,), (64,)]
    params, grads, ms, vs = configs.c5_inputs(13, shapes)
    O = EagerOracle()
    op, og, om, ov = ([O.leaf(a, "f32") for a in arrs] for arrs in (params, grads, ms, vs))

    def dev(arr, shift):
        store = torch.zeros(arr.size + 8, dtype=torch.float32, device="cuda:0")
        view = store[shift:shift + arr.size]
        view.copy_(torch.from_numpy(arr.reshape(-1)).to("cuda:0"))
        return c.from_device_ptr(view.data_ptr(), "f32", arr.shape, keep=store)

    gp = [dev(a, 1 if i == 1 else 0) for i, a in enumerate(params)]   # one parameter is 4-byte aligned only
    gg = [dev(a, 0) for a in grads]
    gm = [dev(a, 2 if i == 2 else 0) for i, a in enumerate(ms)]
    gv = [dev(a, 0) for a in vs]
    for step in (1, 2):
        traces.adam_step(O, op, og, om, ov, step=step)
        traces.adam_step(c, gp, gg, gm, gv, step=step)
        c.barrier()
    assert c.stats()["launches_multi"] == 2
    for a, r in zip(gp + gm + gv, op + om + ov):
        assert_matches(c.fetch(a), r.array, "f32", "adam with unaligned instances")
    c.close()
