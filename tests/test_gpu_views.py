"""GPU parity of the shape operations and of views (paper Section 4.4): the library records forward and backward
sequences of pure operations; the oracle side uses numpy views of shared storage, op by op."""
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


def _data(shape, dtype, seed):
    x = rng.normal_f32(rng.generator(seed), shape, 1.0)
    if dtype == "bf16":
        return rng.to_bf16_bits(x)
    if dtype == "u8":
        return (x > 0).astype(np.uint8) * 7
    if dtype == "i32":
        return (x * 1000).astype(np.int32)
    return x


@pytest.mark.parametrize("dtype", ["f32", "bf16", "u8", "i32"])
@pytest.mark.parametrize("shape", [(3, 4, 5), (7, 33), (2, 3, 4, 6), (129,), (64, 256)])
def test_shape_operations(ctx, dtype, shape):
    a = _data(shape, dtype, 71)
    O = EagerOracle()
    ox, gx = O.leaf(a, dtype), ctx.leaf(a, dtype)
    rank = len(shape)
    cases = []
    for dim in range(rank):
        n = shape[dim]
        cases.append(("narrow", dict(dim=dim, start=n // 3, length=max(1, n // 2))))
    perms = [tuple(reversed(range(rank))), tuple(list(range(1, rank)) + [0])]
    for p in perms:
        cases.append(("permute", dict(perm=p)))
    total = int(np.prod(shape))
    cases.append(("reshape", dict(shape=(total,))))
    if total % 3 == 0:
        cases.append(("reshape", dict(shape=(3, total // 3))))
    outs = [(name, kw, ctx.op(name, gx, **kw)) for name, kw in cases]
    # computed inputs as well: the op then reads a value another kernel produced
    if dtype in ("f32", "bf16"):
        outs += [(name, kw, ctx.op(name, ctx.op("add", gx, gx), **kw)) for name, kw in cases]
    ctx.barrier()
    k = 0
    for name, kw, t in outs:
        src = ox if k < len(cases) else O.op("add", ox, ox)
        ref = O.op(name, src, **kw)
        assert_matches(ctx.fetch(t), ref.array, dtype, f"{name} {kw} {dtype} {shape}", exact=True)
        k += 1
    # update_slice against every narrow
    for dim in range(rank):
        n = shape[dim]
        start, length = n // 3, max(1, n // 2)
        upd_shape = shape[:dim] + (length,) + shape[dim + 1:]
        u = _data(upd_shape, dtype, 72 + dim)
        ref = O.op("update_slice", ox, O.leaf(u, dtype), dim=dim, start=start)
        got = ctx.fetch(ctx.op("update_slice", gx, ctx.leaf(u, dtype), dim=dim, start=start))
        assert_matches(got, ref.array, dtype, f"update_slice dim {dim} {dtype} {shape}", exact=True)


def _paper_example(B, x):
    v = B.view_permute(x, (1, 2, 0))
    B.assign(v, B.op("add", v, B.scalar(42.0)))
    return v


def test_in_place_update_of_a_permuted_view(ctx):
    x0 = rng.normal_f32(rng.generator(73), (2, 3, 4))
    O = EagerOracle()
    ox, gx = O.leaf(x0, "f32"), ctx.leaf(x0, "f32")
    ov, gv = _paper_example(O, ox), _paper_example(ctx, gx)
    assert_matches(ctx.fetch(gx), ox.array, "f32", "base after v.add_(42)", exact=True)
    assert_matches(ctx.fetch(gv), np.ascontiguousarray(ov.array), "f32", "the view", exact=True)
    np.testing.assert_array_equal(ox.array, x0 + np.float32(42))


def test_in_place_update_through_a_narrow_is_written_into_the_base_buffer(ctx):
    import torch

    shape, dim, start, length = (300, 1024), 1, 256, 512
    x0 = rng.normal_f32(rng.generator(74), shape)
    O = EagerOracle()
    ox = O.leaf(x0, "f32")
    xd = torch.from_numpy(x0).cuda()
    gx = ctx.from_torch(xd)
    for step in range(3):
        for B, x in ((O, ox), (ctx, gx)):
            v = B.view_narrow(x, dim, start, length)
            B.assign(v, B.op("mul", B.op("add", v, B.scalar(1.0)), B.scalar(0.5)))
        ctx.barrier()
        assert ctx.device_ptr(gx) == xd.data_ptr()  # the base was updated in its own buffer: only the slice was written
        assert_matches(xd.cpu().numpy(), ox.array, "f32", f"base after step {step}", exact=True)
    st = ctx.stats()
    assert st["outputs_donated"] == 3 and st["compiles"] == 1 and st["cache_hits"] == 2
    want = x0.copy()
    for _ in range(3):
        want[:, start:start + length] = (want[:, start:start + length] + np.float32(1)) * np.float32(0.5)
    np.testing.assert_array_equal(ox.array, want)


def test_views_see_updates_of_their_base_and_of_each_other(ctx):
    x0 = rng.normal_f32(rng.generator(75), (6, 10, 8))
    O = EagerOracle()
    ox, gx = O.leaf(x0, "f32"), ctx.leaf(x0, "f32")
    res = {}
    for name, B, x in (("o", O, ox), ("g", ctx, gx)):
        a = B.view_narrow(x, 1, 2, 5)            # [6, 5, 8]
        b = B.view_permute(a, (2, 0, 1))         # [8, 6, 5]
        c = B.view_narrow(x, 0, 1, 3)            # [3, 10, 8], overlaps a
        B.assign(x, B.op("mul", x, B.scalar(2.0)))
        B.assign(b, B.op("add", b, B.scalar(1.0)))     # through two view operations
        B.assign(c, B.op("neg", c))                    # overlapping view of the same base
        res[name] = (x, a, b, c)
    ctx.barrier()
    for k, what in enumerate(("base", "narrow", "permute of narrow", "overlapping narrow")):
        assert_matches(ctx.fetch(res["g"][k]), np.ascontiguousarray(res["o"][k].array), "f32", what, exact=True)
    want = x0 * np.float32(2)
    want[:, 2:7, :] += np.float32(1)
    want[1:4] *= -1
    np.testing.assert_array_equal(res["o"][0].array, want)


def test_reshape_views(ctx):
    x0 = rng.normal_f32(rng.generator(76), (8, 12))
    O = EagerOracle()
    ox, gx = O.leaf(x0, "f32"), ctx.leaf(x0, "f32")
    for B, x in ((O, ox), (ctx, gx)):
        r = B.view_reshape(x, (4, 24))
        B.assign(r, B.op("sub", r, B.op("row_max", r)))   # rows of the reshaped view
    assert_matches(ctx.fetch(gx), ox.array, "f32", "base after an update through a reshape", exact=True)
    want = x0.reshape(4, 24)
    want = (want - want.max(axis=1, keepdims=True)).reshape(8, 12)
    np.testing.assert_array_equal(ox.array, want)


@pytest.mark.parametrize("mode", ["interpreted", "specialised"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape,dim,start,length", [((64, 256), 1, 64, 128), ((37, 100), 1, 3, 40), ((64, 256), 0, 16, 8),
                                                     ((5, 6, 64), 2, 8, 32), ((300, 1024), 1, 512, 256)])
def test_slices_read_in_place_by_fused_groups(lt, mode, dtype, shape, dim, start, length):
    """A narrow of materialised data feeding elementwise work and a row reduction: read with pitched (or offset) loads
    inside the fused kernel, on the interpreter and on the run-time specialised shells."""
    c = lt.LazyContext(device=0)
    if mode == "interpreted":
        c.set_option("compiled", 0)
    else:
        c.set_option("specialise", 1)
    a = _data(shape, dtype, 77)
    sl_shape = shape[:dim] + (length,) + shape[dim + 1:]
    b = _data(sl_shape, dtype, 78)
    O = EagerOracle()

    def graph(B, x, y):
        s = B.op("narrow", x, dim=dim, start=start, length=length)
        t = B.op("convert", B.op("mul", s, y), dtype="f32")
        return B.op("sub", t, B.op("row_max", t))

    ref = graph(O, O.leaf(a, dtype), O.leaf(b, dtype))
    out = graph(c, c.leaf(a, dtype), c.leaf(b, dtype))
    c.barrier()
    st = c.stats()
    assert st["kernels_launched"] == 1 and st["launches_view"] == 0, (st, c.dump_plan())
    if mode == "specialised" and "specialised at run time" in c.dump_plan() and sl_shape[-1] % 8 == 0 and (start * (2 if dtype == "bf16" else 4)) % 16 == 0:
        assert st["launches_specialised"] == 1, c.dump_plan()
    assert_matches(c.fetch(out), ref.array, "f32", f"in-place slice {shape} {dim} {start} {length} {dtype} {mode}")
    c.close()
