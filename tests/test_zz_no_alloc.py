"""lt_barrier_static_scratch against lt_barrier, through the C ABI, on a GPU.

Some users of the library may not allocate device memory while they run: a control loop with a
latency budget (an allocator call may synchronise the device), a plug-in that owns only the
buffers its host application handed it, a process that starts after another framework has taken
the rest of the GPU.  For them the library has one flush that places the values passed between
its kernels in a fixed device array and writes every result over an input.  The test runs a graph
that needs such in-between values (an unfused RMS-style normalisation, updated in place) through
both flushes and compares them with each other and with the CPU oracle's evaluation of the same
ops, twice in a row because the array keeps the previous call's data.  The file sorts last so that a failure here cannot hide one elsewhere.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

ROWS, COLS = 384, 1000  # 1.5 MB per tensor: ragged rows, several CTAs


def _inputs():
    from workloads import rng

    x = rng.normal_f32(rng.generator(41, 0), (ROWS, COLS), 1.0)
    g = rng.normal_f32(rng.generator(41, 1), (COLS,), 0.1, mean=1.0)
    return x, g


def _record_update(ctx, x, g):
    """x := x * rsqrt(mean(x^2) + eps) * g, recorded op by op; nothing but x stays live."""
    sq = ctx.op("mul", x, x)
    ms = ctx.op("mul", ctx.op("row_sum", sq), ctx.scalar(1.0 / COLS))
    inv = ctx.op("rsqrt", ctx.op("add", ms, ctx.scalar(1e-5)))
    y = ctx.op("mul", ctx.op("mul", x, inv), g)
    ctx.assign(x, y)


def _run(static: bool, steps: int):
    import torch

    import paper_2102_13267_b200 as lt

    ctx = lt.LazyContext(device=0)
    ctx.set_option("fusion", 0)  # one kernel per op: six values travel between kernels
    xh, gh = _inputs()
    xd = torch.from_numpy(xh).cuda()
    gd = torch.from_numpy(gh).cuda()
    x, g = ctx.from_torch(xd), ctx.from_torch(gd)
    outs = []
    for _ in range(steps):
        _record_update(ctx, x, g)
        before = ctx.stats()
        if static:
            ctx.barrier_static_scratch(blocking=True)
        else:
            ctx.barrier(blocking=True)
        after = ctx.stats()
        assert after["temporaries_allocated"] - before["temporaries_allocated"] == 6
        assert after["outputs_donated"] - before["outputs_donated"] == 1
        assert after["outputs_allocated"] == before["outputs_allocated"]
        assert ctx.device_ptr(x) == xd.data_ptr()  # written in place, in the caller's buffer
        outs.append(xd.cpu().numpy().copy())
    ctx.close()
    return outs


def _oracle(steps: int):
    """The same ops, one at a time, on the CPU oracle."""
    from oracle.eager import EagerOracle

    O = EagerOracle()
    xh, gh = _inputs()
    x, g = O.leaf(xh, "f32"), O.leaf(gh, "f32")
    outs = []
    for _ in range(steps):
        _record_update(O, x, g)
        outs.append(O.fetch(x))
    return outs


def test_static_scratch_flush_matches_the_allocating_flush_twice_in_a_row():
    ref = _run(static=False, steps=2)
    got = _run(static=True, steps=2)
    want = _oracle(steps=2)
    for r, g, w in zip(ref, got, want):
        np.testing.assert_allclose(g, r, rtol=1e-5, atol=1e-6)
        assert np.array_equal(g, r)  # same kernels, same order: in fact identical
        np.testing.assert_allclose(g, w, rtol=1e-5, atol=1e-6)  # and both agree with the op-by-op evaluation
        np.testing.assert_allclose(r, w, rtol=1e-5, atol=1e-6)
    assert not np.array_equal(ref[0], ref[1])  # the second step really computed something new


def test_static_scratch_flush_with_clear_first_and_another_current_device_setting():
    """`clear_first` zero-fills the array after the checks and before the kernels; the result is unchanged."""
    import torch

    import paper_2102_13267_b200 as lt

    ctx = lt.LazyContext(device=0)
    ctx.set_option("fusion", 0)
    xh, gh = _inputs()
    xd, gd = torch.from_numpy(xh).cuda(), torch.from_numpy(gh).cuda()
    x, g = ctx.from_torch(xd), ctx.from_torch(gd)
    _record_update(ctx, x, g)
    ctx.barrier_static_scratch(blocking=True, clear_first=True)
    np.testing.assert_allclose(xd.cpu().numpy(), _oracle(steps=1)[0], rtol=1e-5, atol=1e-6)
    ctx.close()


def test_static_scratch_flush_refuses_what_it_cannot_place():
    import torch

    import paper_2102_13267_b200 as lt

    ctx = lt.LazyContext(device=0)
    xd = torch.ones(64, 64, device="cuda")
    x = ctx.from_torch(xd)
    y = ctx.op("mul", x, x)  # a fresh result: it would need new memory
    with pytest.raises(lt.LazyTensorError) as err:
        ctx.barrier_static_scratch(blocking=True)
    assert err.value.status == lt.STATUS_NAMES.index("LT_ERR_UNSUPPORTED")
    assert np.array_equal(ctx.fetch(y), np.ones((64, 64), np.float32))  # still pending; lt_fetch flushes it

    # temporaries beyond the array's size
    ctx.set_option("fusion", 0)
    n = 3 * 1024 * 1024  # 12 MB per value; the chain below passes three of them between kernels
    bd = torch.ones(n, device="cuda")
    b = ctx.from_torch(bd)
    ctx.assign(b, ctx.op("mul", ctx.op("add", ctx.op("mul", b, b), b), ctx.op("neg", b)))
    with pytest.raises(lt.LazyTensorError) as err:
        ctx.barrier_static_scratch(blocking=True)
    assert err.value.status == lt.STATUS_NAMES.index("LT_ERR_UNSUPPORTED")
    assert "static scratch" in str(err.value)
    ctx.barrier(blocking=True)
    assert float(bd[0]) == -2.0
    ctx.close()


def test_static_scratch_holds_the_partials_of_a_reduction_kernel():
    """A whole-tensor reduction runs in two stages through a temporary: with the allocation-free flush that temporary
    lives in the fixed array too."""
    import torch

    import paper_2102_13267_b200 as lt
    from oracle.eager import EagerOracle

    ctx = lt.LazyContext(device=0)
    xh, _ = _inputs()
    xd = torch.from_numpy(xh).cuda()
    x = ctx.from_torch(xd)
    O = EagerOracle()
    ox = O.leaf(xh, "f32")
    for B, t in ((O, ox), (ctx, x)):
        B.assign(t, B.op("sub", t, B.op("all_max", t)))
    ctx.barrier_static_scratch(blocking=True)
    assert ctx.device_ptr(x) == xd.data_ptr() and ctx.stats()["launches_reduce"] == 1
    np.testing.assert_allclose(xd.cpu().numpy(), ox.array, rtol=1e-5, atol=1e-6)
    ctx.close()
