"""Trace matching on the GPU: steps that repeat the previous step's calls run on the logged plan without the graph
being built, and every step's values must still be what the CPU oracle computes -- with new inputs, new run-time
scalars, new random seeds and in-place updates bound through the matched path."""
import numpy as np
import pytest

from helpers import assert_matches
from oracle.eager import EagerOracle
from workloads import configs, rng, traces

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lt():
    import paper_2102_13267_b200 as lt
    return lt


def test_new_inputs_and_scalars_every_step(lt):
    c, O = lt.LazyContext(device=0), EagerOracle()
    shape = (257, 1000)
    w = rng.normal_f32(rng.generator(301), shape)
    gw, ow = c.leaf(w, "f32"), O.leaf(w, "f32")
    for step in range(8):
        x = rng.normal_f32(rng.generator(310 + step), shape)
        outs = []
        for B, wt in ((O, ow), (c, gw)):
            xt = B.leaf(x, "f32")                                     # a leaf made inside the trace
            y = B.op("tanh", B.op("mul", B.op("add", xt, wt), B.scalar(0.25 * (step + 1))))
            r = B.op("row_sum", B.op("mul", y, y))           # (squares: no cancellation in the sums)
            outs.append((y, r))
        (oy, orow), (gy, grow) = outs
        assert_matches(c.fetch(grow), orow.array, "f32", f"row sums, step {step}")  # the fetch flushes the matched trace
        assert_matches(c.fetch(gy), oy.array, "f32", f"values, step {step}")
        del outs, gy, grow
    st = c.stats()
    assert st["traces_matched"] >= 3 and st["compiles"] <= 2, st  # (the first step has no temporaries of an earlier one to drop)
    c.close()


def test_dropout_with_a_new_seed_every_step(lt):
    """The seed and offset of the random bits are run-time values: they differ every step and the trace still matches."""
    c, O = lt.LazyContext(device=0), EagerOracle()
    shape = (96, 1024)
    x, h, g, b = configs.c3_inputs(320, shape)
    G = [c.leaf(a, d) for a, d in ((x, "bf16"), (h, "bf16"), (g, "f32"), (b, "f32"))]
    R = [O.leaf(a, d) for a, d in ((x, "bf16"), (h, "bf16"), (g, "f32"), (b, "f32"))]
    for step in range(6):
        kw = dict(shape=shape, p=0.1, eps=1e-5, seed=1000 + 17 * step, offset=step * (1 << 20))
        zr, kr = traces.residual_dropout_layernorm(O, *R, **kw)
        z, k = traces.residual_dropout_layernorm(c, *G, **kw)
        c.barrier()
        assert_matches(c.fetch(k), kr.array, "u8", f"mask, step {step}")
        assert_matches(c.fetch(z), zr.array, "bf16", f"z, step {step}")
        del z, k
    st = c.stats()
    assert st["traces_matched"] >= 2 and st["compiles"] <= 2, st
    c.close()


def test_in_place_updates_through_matched_traces(lt):
    """Momentum SGD on a few tensors, updated in place for 30 steps; a tensor that aliases a parameter appears for
    a while in the middle, during which nothing may be written into that parameter's buffer."""
    c, O = lt.LazyContext(device=0), EagerOracle()
    shapes = [(64, 3, 3, 3), (64,), (1000, 96), (17,)]
    host = [[rng.normal_f32(rng.generator(330 + 10 * j + i), s, 0.1) for i, s in enumerate(shapes)] for j in range(3)]
    gp, gg, gm = ([c.leaf(a, "f32") for a in arrs] for arrs in host)
    op, og, om = ([O.leaf(a, "f32") for a in arrs] for arrs in host)
    alias = {}
    for step in range(30):
        for B, P, Gr, M in ((O, op, og, om), (c, gp, gg, gm)):
            if step == 12:
                alias[B] = B.op("add", P[2], B.scalar(0.0))
                B.assign(alias[B], P[2])           # a second tensor naming P[2]'s value
            if step == 20:
                B.release(alias.pop(B))
            mom, lr = B.scalar(0.9), B.scalar(0.05 / (1 + step))
            for p, g, m in zip(P, Gr, M):
                m_new = B.op("add", B.op("mul", m, mom), g)
                B.assign(m, m_new)
                B.assign(p, B.op("sub", p, B.op("mul", m_new, lr)))
        c.barrier()
        if step % 7 == 0 or step in (12, 13, 20, 21):
            for a, r in zip(gp + gm, op + om):
                assert_matches(c.fetch(a), r.array, "f32", f"step {step}")
            if c in alias:
                assert_matches(c.fetch(alias[c]), alias[O].array, "f32", f"alias, step {step}")
    for a, r in zip(gp + gm, op + om):
        assert_matches(c.fetch(a), r.array, "f32", "final")
    st = c.stats()
    assert st["traces_matched"] >= 12 and st["compiles"] == 2, st  # with and without the alias; steps 12 and 20 differ from their logs in the first call
    c.close()


def test_matching_off_gives_the_same_bits(lt):
    results = []
    for on in (1, 0):
        c = lt.LazyContext(device=0)
        c.set_option("trace_match", on)
        x = c.leaf(rng.normal_f32(rng.generator(340), (300, 512)), "f32")
        acc = c.leaf(np.zeros((300, 512), np.float32), "f32")
        for step in range(6):
            c.assign(acc, c.op("add", c.op("mul", acc, c.scalar(0.5)), c.op("exp", c.op("mul", x, c.scalar(0.1 * step)))))
            c.barrier()
        results.append(c.fetch(acc))
        assert (c.stats()["traces_matched"] > 0) == bool(on)
        c.close()
    np.testing.assert_array_equal(results[0], results[1])


def test_adam_recorded_in_batches_matches_the_oracle(lt):
    """One lt_op_many call per parameter and step (the update's thirteen operations and three in-place assignments)."""
    from workloads import configs

    class Names:
        pass

    batch, refs = lt.Batch(), Names()
    b_in = [batch.input() for _ in range(4)]
    names = ("beta1", "one_minus_beta1", "beta2", "one_minus_beta2", "sqrt_bc2", "eps", "step_size")
    for n in names:
        setattr(refs, n, batch.input())
    traces.adam_update(batch, *b_in, refs)
    shapes = [(64, 3, 7, 7), (64,), (256, 64, 1, 1), (1000, 96), (1000,)]
    p, g, m, v = configs.c5_inputs(350, shapes)
    c, O = lt.LazyContext(device=0), EagerOracle()
    gp, gg, gm, gv = ([c.leaf(a, "f32") for a in arrs] for arrs in (p, g, m, v))
    op, og, om, ov = ([O.leaf(a, "f32") for a in arrs] for arrs in (p, g, m, v))
    for step in range(1, 13):
        traces.adam_step(O, op, og, om, ov, step=step)
        s = traces.AdamScalars(c, step=step)
        for t in zip(gp, gg, gm, gv):
            c.record(batch, [*t, *(getattr(s, n) for n in names)])
        c.barrier()
    for got, ref in zip(gp + gm + gv, op + om + ov):
        assert_matches(c.fetch(got), ref.array, "f32", "Adam recorded in batches")
    st = c.stats()
    assert st["compiles"] == 1 and st["cache_hits"] == 11 and st["launches_multi"] == 12 and st["traces_matched"] >= 9, st
    c.close()
