"""Run-time specialisation on the GPU: programs without a kernel in the build-time table get the same shells
instantiated at run time; results must match the oracle exactly as the interpreter's and the table's do."""
import time

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


def _bias_tanh_scale(B, x, bias, s):
    """An elementwise group that is not in the table: tanh(x + bias) * s - x."""
    t = B.op("tanh", B.op("add", x, bias))
    return B.op("sub", B.op("mul", t, s), x)


def _row_normalise(B, z):
    """A row group that is not in the table: |z - max| / (sum |z - max| + 3)."""
    d = B.op("abs", B.op("sub", z, B.op("row_max", z)))
    return B.op("div", d, B.op("add", B.op("row_sum", d), B.scalar(3.0)))


def _needs_specialiser(ctx):
    if "specialised at run time" not in ctx.dump_plan():
        pytest.skip("the run-time compiler library is not installed")


@pytest.mark.parametrize("shape", [(64, 256), (300, 1024), (7, 2048), (5, 40)])
def test_specialised_at_planning_time(lt, shape):
    c = lt.LazyContext(device=0)
    c.set_option("specialise", 1)
    g = rng.generator(81)
    x, bias, z = rng.normal_f32(g, shape), rng.normal_f32(g, (shape[-1],)), rng.normal_f32(g, shape)
    O = EagerOracle()
    ref_e = _bias_tanh_scale(O, O.leaf(x, "f32"), O.leaf(bias, "f32"), O.scalar(0.75))
    ref_r = _row_normalise(O, O.leaf(z, "f32"))
    out_e = _bias_tanh_scale(c, c.leaf(x, "f32"), c.leaf(bias, "f32"), c.scalar(0.75))
    c.barrier()
    _needs_specialiser(c)
    out_r = _row_normalise(c, c.leaf(z, "f32"))
    c.barrier()
    st = c.stats()
    assert st["kernels_launched"] == 2 and st["programs_specialised"] == 2
    assert st["launches_specialised"] == 2 and st["launches_compiled"] == 2, (st, c.dump_plan())
    assert_matches(c.fetch(out_e), ref_e.array, "f32", f"specialised elementwise {shape}")
    assert_matches(c.fetch(out_r), ref_r.array, "f32", f"specialised row {shape}")
    c.close()


def test_specialised_in_the_background_takes_over_mid_stream(lt):
    c = lt.LazyContext(device=0)  # default mode: a worker thread, after the plan has run three times
    shape = (512, 1024)
    g = rng.generator(82)
    x, bias = rng.normal_f32(g, shape), rng.normal_f32(g, (shape[-1],))
    O = EagerOracle()
    ref = _bias_tanh_scale(O, O.leaf(x, "f32"), O.leaf(bias, "f32"), O.scalar(0.75)).array
    gx, gb = c.leaf(x, "f32"), c.leaf(bias, "f32")
    deadline = time.time() + 60
    first = None
    flushes = 0
    while time.time() < deadline:
        out = _bias_tanh_scale(c, gx, gb, c.scalar(0.75))
        c.barrier()
        flushes += 1
        got = c.fetch(out)
        assert_matches(got, ref, "f32", f"flush {flushes}")
        if flushes == 1:
            _needs_specialiser(c)
            first = got
        if c.stats()["launches_specialised"] >= 2:
            break
        time.sleep(0.05)
    st = c.stats()
    assert st["launches_specialised"] >= 2, (st, c.dump_plan())
    assert st["compiles"] == 1 and st["programs_specialised"] == 1 and st["launches_compiled"] == st["launches_specialised"]
    assert st["launches_elementwise"] == flushes  # the interpreter served the flushes before the kernel was there
    np.testing.assert_allclose(got, first, rtol=1e-5, atol=1e-6)
    c.close()


def test_unlisted_long_rows_run_split_until_their_kernel_is_built(lt):
    """Default mode: a long-row group that is not in the table runs with its reductions as kernels of their own while
    the specialiser builds the fused kernel in the background, then fused -- every flush against the oracle."""
    c = lt.LazyContext(device=0)
    z = rng.normal_f32(rng.generator(85), (64, 16384))
    O = EagerOracle()
    ref = _row_normalise(O, O.leaf(z, "f32")).array
    gz = c.leaf(z, "f32")
    deadline = time.time() + 90
    flushes = 0
    while time.time() < deadline:
        out = _row_normalise(c, gz)
        c.barrier()
        flushes += 1
        assert_matches(c.fetch(out), ref, "f32", f"flush {flushes}")
        if flushes == 1:
            _needs_specialiser(c)
            assert c.stats()["launches_reduce"] == 2  # the two long reductions on their own
        if c.stats()["launches_specialised"] >= 2:
            break
        time.sleep(0.05)
    st = c.stats()
    # (the elementwise pieces of the split variant may have been handed to the specialiser as well)
    assert st["launches_specialised"] >= 2 and st["compiles"] == 1 and st["programs_specialised"] >= 1, (st, c.dump_plan())
    split_flushes = st["launches_reduce"] // 2
    assert 3 <= split_flushes < flushes and st["launches_reduce"] == 2 * split_flushes  # nothing split once the kernel is there
    assert st["launches_row"] == flushes - split_flushes
    c.close()


def test_specialised_long_rows_and_multi_tensor(lt):
    c = lt.LazyContext(device=0)
    c.set_option("specialise", 1)
    z = rng.normal_f32(rng.generator(83), (20, 16384))
    O = EagerOracle()
    ref = _row_normalise(O, O.leaf(z, "f32"))
    out = _row_normalise(c, c.leaf(z, "f32"))
    c.barrier()
    _needs_specialiser(c)
    st = c.stats()
    assert st["launches_row"] == 1 and st["launches_reduce"] == 0 and st["launches_specialised"] == 1
    assert_matches(c.fetch(out), ref.array, "f32", "specialised long rows")
    # the same program on the CTA-per-row kernel, and on every cluster size of the cluster kernel
    for cluster in (1, 2, 4, 8):
        k = lt.LazyContext(device=0)
        k.set_option("specialise", 1)
        k.set_option("debug.cluster", cluster)
        got = _row_normalise(k, k.leaf(z, "f32"))
        k.barrier()
        assert k.stats()["launches_specialised"] == 1
        assert_matches(k.fetch(got), ref.array, "f32", f"specialised long rows, cluster {cluster}")
        k.close()
    # many small tensors, one program that is not in the table: p := p * 0.99 - g * lr, in place
    shapes = [(64, 3, 7, 7), (64,), (1000,), (256, 64), (128,)]
    host = [[rng.normal_f32(rng.generator(84 + k), s, 0.1) for s in shapes] for k in range(2)]
    op, og = ([O.leaf(a, "f32") for a in arrs] for arrs in host)
    gp, gg = ([c.leaf(a, "f32") for a in arrs] for arrs in host)
    for B, P, G in ((O, op, og), (c, gp, gg)):
        decay, lr = B.scalar(0.99), B.scalar(0.05)
        for p, g in zip(P, G):
            B.assign(p, B.op("sub", B.op("mul", p, decay), B.op("mul", g, lr)))
    before = c.stats()["launches_specialised"]
    c.barrier()
    st = c.stats()
    assert st["launches_multi"] == 1 and st["launches_specialised"] == before + 1, (st, c.dump_plan())
    for a, r in zip(gp, op):
        assert_matches(c.fetch(a), r.array, "f32", "specialised multi-tensor", exact=True)
    c.close()
