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
    for shape in [(4, 8), (3, 40), (2, 3, 100), (5, 1), (2, 2048), (1, 64), (1, 1), (64,), (1, 9000)]:
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
EXACT_UNARY = ["relu", "abs", "neg", "square"]
ANY_UNARY = ["tanh", "relu", "abs", "neg", "sigmoid", "square"]


def _random_graph(B, g, leaves, n_ops, exact_ops_only=False):
    """Issues the same random op sequence on backend B; returns the values that stay live.  With
    `exact_ops_only` the sequence holds only ops whose binary32 result is fixed by IEEE 754 (one correctly
    rounded operation each: no transcendental, no reduction, whose summation order is free)."""
    vals = list(leaves)
    unary = EXACT_UNARY if exact_ops_only else ANY_UNARY
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
            vals.append(B.op(unary[g.integers(0, len(unary))], x))
        elif kind == 8:
            name = ["row_sum", "row_max"][g.integers(0, 2)]
            vals.append(B.op("row_max" if exact_ops_only else name, x))
        else:
            m = B.op("gt", x, B.scalar(0.0))
            vals.append(B.op("where", m, x, full[g.integers(0, len(full))]))
    n_keep = int(g.integers(1, 4))
    return vals[-n_keep:]


class _Tracked:
    """An oracle value with a bound on how far a binary32 evaluation of the same ops may be from it."""

    def __init__(self, t, err, undecided=None):
        self.t, self.err, self.undecided = t, err, undecided

    @property
    def shape(self):
        return self.t.shape


class BoundingOracle:
    """Runs the eager oracle and propagates, per element, a running bound on the absolute difference an
    evaluation may show that performs every op in binary32 with these per-op errors: + - * and square correctly
    rounded (u = 2^-24 relative), tanh within 4u and sigmoid within 8u of the exact function of its (already
    perturbed) argument, a row sum accumulated in binary32 in any order ((log2 n + 8) u sum|x|), max / relu /
    abs / neg / row_max without rounding.  A comparison against zero whose operand lies within its own bound of
    zero may go either way; `where` then takes the distance between its two branches into the bound."""

    U = 2.0 ** -24

    def __init__(self):
        self.O = EagerOracle()

    def leaf(self, a, dtype):
        t = self.O.leaf(a, dtype)
        return _Tracked(t, np.zeros(t.shape))

    def scalar(self, v, dtype="f32"):
        return self.O.scalar(v, dtype)

    @staticmethod
    def _ve(x):
        if isinstance(x, _Tracked):
            return x.t.array.astype(np.float64), x.err
        return np.float64(np.float32(x.value)), np.float64(0.0)

    def op(self, name, *ins):
        u = self.U
        raw = [x.t if isinstance(x, _Tracked) else x for x in ins]
        out = self.O.op(name, *raw)
        r = np.abs(out.array.astype(np.float64))
        with np.errstate(all="ignore"):
            if name in ("add", "sub"):
                (a, ea), (b, eb) = self._ve(ins[0]), self._ve(ins[1])
                e = ea + eb
                e = e + u * (r + e)
            elif name == "mul":
                (a, ea), (b, eb) = self._ve(ins[0]), self._ve(ins[1])
                e = np.abs(a) * eb + np.abs(b) * ea + ea * eb
                e = e + u * (r + e)
            elif name == "max":
                e = np.maximum(*np.broadcast_arrays(self._ve(ins[0])[1], self._ve(ins[1])[1]))
            elif name in ("relu", "abs", "neg"):
                e = ins[0].err
            elif name == "square":
                a, ea = self._ve(ins[0])
                e = 2 * np.abs(a) * ea + ea * ea
                e = e + u * (r + e)
            elif name == "tanh":
                e = ins[0].err + 4 * u * (r + ins[0].err)
            elif name == "sigmoid":
                e = ins[0].err / 4 + 8 * u * (r + ins[0].err)
            elif name == "row_sum":
                a, ea = self._ve(ins[0])
                n = a.shape[-1]
                mag = (np.abs(a) + ea).sum(axis=-1, keepdims=True)
                e = ea.sum(axis=-1, keepdims=True) + (np.ceil(np.log2(max(n, 2))) + 8) * u * mag
            elif name == "row_max":
                e = ins[0].err.max(axis=-1, keepdims=True)
            elif name == "gt":
                a, ea = self._ve(ins[0])
                return _Tracked(out, np.zeros(out.shape), undecided=np.abs(a) <= ea)
            elif name == "where":
                m, x, y = ins
                (a, ea), (b, eb) = self._ve(x), self._ve(y)
                a, b, ea, eb, mm, und = np.broadcast_arrays(a, b, ea, eb, m.t.array != 0, m.undecided)
                e = np.where(mm, ea, eb)
                e = np.where(und, np.abs(a - b) + ea + eb, e)
            else:
                raise AssertionError(name)
        e = np.where(np.isfinite(e), e, np.inf)
        return _Tracked(out, np.broadcast_to(e, out.shape).astype(np.float64))


@pytest.mark.parametrize("seed", range(12))
@pytest.mark.parametrize("fusion", [1, 0])
def test_random_graphs(lt, seed, fusion):
    """Random graphs with transcendentals and reductions: the stated binary32 tolerance (rel 1e-5, abs 1e-6) plus
    what the graph itself amplifies, bounded op by op alongside the oracle (see BoundingOracle)."""
    shape = [(6, 40), (3, 17), (2, 4, 64), (5, 256)][seed % 4]
    gi = rng.generator(100 + seed)
    arrays = [rng.normal_f32(gi, shape, 1.0) for _ in range(3)] + [rng.normal_f32(gi, (shape[-1],), 1.0)]
    c = lt.LazyContext(device=0)
    c.set_option("fusion", fusion)
    O = BoundingOracle()
    ref = _random_graph(O, rng.generator(500 + seed), [O.leaf(a, "f32") for a in arrays], 14)
    got = _random_graph(c, rng.generator(500 + seed), [c.leaf(a, "f32") for a in arrays], 14)
    c.barrier()
    for k, (r, t) in enumerate(zip(ref, got)):
        a, b = c.fetch(t).astype(np.float64), r.t.array.astype(np.float64)
        assert a.shape == b.shape
        np.testing.assert_array_equal(np.isnan(a), np.isnan(b), err_msg=f"seed {seed} output {k}: NaN positions")
        fin = np.isfinite(b) & np.isfinite(r.err)
        np.testing.assert_array_equal(a[~fin & ~np.isnan(b) & np.isfinite(r.err)], b[~fin & ~np.isnan(b) & np.isfinite(r.err)])
        bound = 1e-6 + 1e-5 * np.abs(b) + r.err
        bad = fin & (np.abs(a - b) > bound)
        assert not bad.any(), (f"seed {seed} output {k}: {bad.sum()} of {bad.size} outside the bound; worst "
                               f"{np.nanmax(np.where(fin, np.abs(a - b) - bound, -np.inf))}")
        # the propagated part stays a modest multiple of the base tolerance on most elements: the check has teeth
        assert np.median(r.err[fin] / (1e-6 + 1e-5 * np.abs(b[fin]))) < 50 if fin.any() else True
    c.close()


@pytest.mark.parametrize("seed", range(8))
@pytest.mark.parametrize("fusion", [1, 0])
def test_random_graphs_of_exactly_rounded_ops_are_bit_identical(lt, seed, fusion):
    """Graphs of + - * max relu abs neg square where row_max only: every op has one correctly rounded binary32
    result, so with ieee=1 the fused kernels must reproduce the op-by-op evaluation bit for bit."""
    shape = [(6, 40), (3, 17), (2, 4, 64), (5, 256)][seed % 4]
    gi = rng.generator(300 + seed)
    arrays = [rng.normal_f32(gi, shape, 1.0) for _ in range(3)] + [rng.normal_f32(gi, (shape[-1],), 1.0)]
    c = lt.LazyContext(device=0)
    c.set_option("fusion", fusion)
    c.set_option("ieee", 1)
    O = EagerOracle()
    ref = _random_graph(O, rng.generator(700 + seed), [O.leaf(a, "f32") for a in arrays], 14, exact_ops_only=True)
    got = _random_graph(c, rng.generator(700 + seed), [c.leaf(a, "f32") for a in arrays], 14, exact_ops_only=True)
    c.barrier()
    for k, (r, t) in enumerate(zip(ref, got)):
        assert_matches(c.fetch(t), r.array, "f32", f"exact seed {seed} output {k}", exact=True)
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
