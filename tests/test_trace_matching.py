"""Trace matching (host logic, no GPU): a trace that repeats the previous one call by call is bound to that one's
plan without being built; anything else is rebuilt on the same handles and gives what plain recording gives.

The check is differential: the same sequence of API calls is made on a context with the option on and on one with
it off, and after every barrier the two must agree on what was planned, what was launched, and what every live
tensor is.  Paper section 7 (future work: the cost of re-tracing) is what the feature answers; the paper fixes no
behaviour here beyond "same results as tracing", which is what is tested.
"""
import os
import random
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import paper_2102_13267_b200 as lt  # noqa: E402


def fake(ctx, shape, dtype="f32", base=[1 << 34]):
    base[0] += 1 << 28
    return ctx.from_device_ptr(base[0], dtype, shape)


def pair():
    on, off = lt.LazyContext(device=None), lt.LazyContext(device=None)
    off.set_option("trace_match", 0)
    return on, off


def delta(ctx, before):
    after = ctx.stats()
    return {k: after[k] - before[k] for k in ("compiles", "cache_hits", "kernels_launched", "barriers", "nodes_recorded")}


def adam_like(ctx, P, G, M, lr, steps_done):
    """An in-place update of three tensors per parameter, temporaries dropped as Python drops them."""
    b1, omb1 = ctx.scalar(0.9), ctx.scalar(0.1)
    step = ctx.scalar(lr / (1 + steps_done))
    for p, g, m in zip(P, G, M):
        m_new = ctx.op("add", ctx.op("mul", m, b1), ctx.op("mul", g, omb1))
        ctx.assign(m, m_new)
        ctx.assign(p, ctx.op("sub", p, ctx.op("mul", m_new, step)))


def test_repeated_trace_is_matched_and_counts_as_a_cache_hit():
    on, off = pair()
    for ctx in (on, off):
        P = [fake(ctx, (64, 64)) for _ in range(3)]
        G = [fake(ctx, (64, 64)) for _ in range(3)]
        M = [fake(ctx, (64, 64)) for _ in range(3)]
        seen = []
        for k in range(6):
            before = ctx.stats()
            adam_like(ctx, P, G, M, 1e-3, k)
            ctx.barrier()
            seen.append((delta(ctx, before), ctx.dump_plan()))
        ctx.seen = seen
        ctx.keep = (P, G, M)
    assert on.seen == off.seen
    assert [d["compiles"] for d, _ in on.seen] == [1, 0, 0, 0, 0, 0]
    st = on.stats()
    assert st["traces_matched"] == 4 and st["traces_diverged"] == 0  # the first trace is built, the second logged against it
    assert off.stats()["traces_matched"] == 0
    assert "donated" in on.seen[-1][1]  # the updates are written in place in the matched flushes too


def test_divergence_rebuilds_the_prefix_on_the_same_handles():
    on, off = pair()
    out = {}
    for ctx in (on, off):
        x, y = fake(ctx, (32, 128)), fake(ctx, (32, 128))
        texts = []
        for k in range(5):
            a = ctx.op("add", x, y)
            b = ctx.op("mul", a, ctx.scalar(3.0))
            if k == 3:  # differs after two matched calls and a scalar: `a` and `b` must still be usable
                c_ = ctx.op("sub", b, a)
                texts.append(ctx.dump_ir())
            else:
                c_ = ctx.op("exp", b)
            d = ctx.op("add", c_, a)
            before = ctx.stats()
            ctx.barrier()
            texts.append((delta(ctx, before), ctx.dump_plan(), d.shape, d.dtype, ctx.is_materialised(d), ctx.is_materialised(a)))
            del a, b, c_, d
        out[ctx] = texts
    assert out[on] == out[off]
    assert on.stats()["traces_diverged"] == 2  # step 3 leaves the log of steps 0-2, step 4 the log of step 3
    assert on.stats()["traces_matched"] >= 1


@pytest.mark.parametrize("variant", ["static_scalar", "operand", "shorter", "longer", "release_order", "alias", "dtype", "early_barrier"])
def test_every_kind_of_difference_is_noticed(variant):
    on, off = pair()
    out = {}
    for ctx in (on, off):
        x, y, z = fake(ctx, (16, 64)), fake(ctx, (16, 64)), fake(ctx, (16, 64))
        xb = fake(ctx, (16, 64), "bf16")
        x2 = ctx.from_device_ptr(ctx.device_ptr(x), "f32", (16, 64))  # another tensor over x's memory
        log = []
        for k in range(6):
            odd = k == 4  # (the first trace has no releases of an earlier step's tensors, so the second one differs from it)
            s = ctx.scalar(0.0 if (odd and variant == "static_scalar") else 2.0 + k)
            lhs = y if (odd and variant == "operand") else (xb if (odd and variant == "dtype") else x)
            if lhs is xb:
                lhs = ctx.op("convert", lhs, dtype="f32")
            a = ctx.op("mul", lhs, s)
            b = ctx.op("add", a, z)
            if odd and variant == "early_barrier":
                ctx.barrier()
            c_ = ctx.op("tanh", b) if not (odd and variant == "shorter") else b
            if odd and variant == "longer":
                c_ = ctx.op("neg", c_)
            if odd and variant == "release_order":
                ctx.release(b)
                ctx.release(a)
            elif variant == "release_order":
                ctx.release(a)
                ctx.release(b)
            d = ctx.op("add", c_, x2 if (odd and variant == "alias") else x)
            before = ctx.stats()
            ctx.barrier()
            log.append((delta(ctx, before), ctx.dump_plan(), d.shape, ctx.is_materialised(d)))
            del s, a, b, c_, d
        out[ctx] = log
    assert out[on] == out[off]
    # (a difference in the very first call leaves nothing to rebuild and is not counted as a divergence)
    assert on.stats()["traces_matched"] >= 1 and (on.stats()["traces_diverged"] >= 1 or variant == "static_scalar")


def test_in_place_result_is_not_written_over_memory_another_tensor_names():
    """The logged plan writes p's update into p's buffer.  In a later step a second tensor names that buffer: the
    matched barrier must notice (Section 4.3: donation only when nothing else names the buffer) and plan again."""
    on, off = pair()
    out = {}
    for ctx in (on, off):
        p, g = fake(ctx, (8, 256)), fake(ctx, (8, 256))
        log, extra = [], None
        for k in range(5):
            if k == 3:
                extra = ctx.op("add", p, ctx.scalar(0.0))  # flushed below: `extra` then owns a buffer of its own
                ctx.barrier()
                alias = ctx.from_device_ptr(ctx.device_ptr(g), "f32", (8, 256))
                log.append(ctx.is_materialised(extra))
                del alias
            q = ctx.op("sub", p, ctx.op("mul", g, ctx.scalar(0.1 * (k + 1))))
            ctx.assign(p, q)
            del q
            before = ctx.stats()
            ctx.barrier()
            log.append((delta(ctx, before), ctx.dump_plan()))
        out[ctx] = log
    assert out[on] == out[off]
    # two handles over one leaf: the receiver is not alone, nothing may be written in place
    for ctx in (on, off):
        p = fake(ctx, (8, 256))
        p_again = None
        plans = []
        for k in range(4):
            if k == 2:
                p_again = ctx.op("add", p, ctx.scalar(0.0))
                ctx.assign(p_again, p)  # p_again now names p's leaf as well
            ctx.assign(p, ctx.op("mul", p, ctx.scalar(0.5)))
            ctx.barrier()
            plans.append("donated" in ctx.dump_plan())
        out[ctx] = plans
    assert out[on] == out[off]


def test_tensor_info_of_matched_results_needs_no_rebuild():
    ctx = lt.LazyContext(device=None)
    x = fake(ctx, (4, 5, 6), "bf16")
    for k in range(4):
        y = ctx.op("convert", ctx.op("relu", x), dtype="f32")
        r = ctx.op("row_sum", y)
        assert y.shape == (4, 5, 6) and y.dtype == "f32" and r.shape == (4, 5, 1)
        assert not ctx.is_materialised(r)
        ctx.barrier()
        assert ctx.is_materialised(r)
        del y, r
    st = ctx.stats()
    assert st["traces_matched"] == 2 and st["traces_diverged"] == 0
    ctx.close()


def test_replay_after_a_matched_flush():
    on, off = pair()
    out = {}
    for ctx in (on, off):
        p, g = fake(ctx, (128,)), fake(ctx, (128,))
        lr = ctx.scalar(0.5, dynamic=True)
        for k in range(3):
            ctx.assign(p, ctx.op("sub", p, ctx.op("mul", g, lr)))
            ctx.barrier()
        ctx.scalar_set(lr, 0.25)
        before = ctx.stats()
        ctx.replay()
        ctx.replay()
        after = ctx.stats()
        out[ctx] = (after["replays"] - before["replays"], after["kernels_launched"] - before["kernels_launched"], ctx.replay_slots())
    assert out[on] == out[off] == (2, 2, 1)
    assert on.stats()["traces_matched"] == 1


def test_scalars_that_outlive_the_trace_and_leaves_made_inside_it():
    on, off = pair()
    out = {}
    for ctx in (on, off):
        x = fake(ctx, (64,))
        log, kept = [], []
        for k in range(6):
            fresh = fake(ctx, (64,))                  # a new input every step, as a data loader gives
            s = ctx.scalar(1.5 + k)
            kept.append(s)                            # still alive after the barrier
            y = ctx.op("mul", ctx.op("add", x, fresh), s)
            z = ctx.op("add", y, kept[0])             # from the second step on: a scalar from an earlier trace
            before = ctx.stats()
            ctx.barrier()
            log.append((delta(ctx, before), ctx.dump_plan(), ctx.is_materialised(y), ctx.is_materialised(z)))
            w = ctx.op("mul", kept[-1], kept[-1]) if False else None
            del fresh, y, z, w
        out[ctx] = log
    assert out[on] == out[off]
    assert on.stats()["traces_matched"] >= 2


def test_option_changes_and_views_fall_back_to_plain_recording():
    ctx = lt.LazyContext(device=None)
    x = fake(ctx, (32, 32))
    for k in range(3):
        y = ctx.op("exp", x)
        ctx.barrier()
        del y
    assert ctx.stats()["traces_matched"] == 1
    ctx.set_option("fusion", 0)                      # the logged plan was made with fusion on
    for k in range(3):
        y = ctx.op("neg", ctx.op("exp", x))
        ctx.barrier()
        del y
    assert "2 launches" in ctx.dump_plan() and ctx.stats()["traces_matched"] == 3  # not the first of the three: its plan is new
    v = ctx.view_narrow(x, 0, 0, 8)                   # a live view: its base's updates are recorded at the barrier
    matched = ctx.stats()["traces_matched"]
    for k in range(3):
        ctx.assign(x, ctx.op("neg", x))
        ctx.barrier()
    assert ctx.stats()["traces_matched"] == matched
    del v
    ctx.close()


def test_random_programs_agree_with_plain_recording():
    """Random straight-line programs over a pool of tensors, repeated with random mutations (another op, another
    operand, a dropped or added call, an in-place update, a release moved) for many steps on both contexts."""
    rng = random.Random(20260117)
    unary, binary = ["exp", "neg", "tanh", "relu", "abs"], ["add", "sub", "mul", "max"]
    matched = diverged = 0
    for trial in range(60):
        n_ops = rng.randint(3, 14)
        base = []
        for i in range(n_ops):
            kind = rng.choice(["u", "b", "b", "s", "a"])
            base.append((kind, rng.choice(unary if kind == "u" else binary), rng.random(), rng.random(), rng.random()))
        on, off = pair()
        results = {}
        for ctx in (on, off):
            r2 = random.Random(trial)
            leaves = [fake(ctx, (8, 32)) for _ in range(3)]
            log = []
            for step in range(12):
                prog = list(base)
                if r2.random() < 0.3:  # mutate this step only
                    j = r2.randrange(len(prog))
                    what = r2.choice(["op", "drop", "dup", "operand"])
                    if what == "op":
                        prog[j] = (prog[j][0], r2.choice(unary if prog[j][0] == "u" else binary), *prog[j][2:])
                    elif what == "drop":
                        prog.pop(j)
                    elif what == "dup":
                        prog.insert(j, prog[j])
                    else:
                        prog[j] = (*prog[j][:2], r2.random(), r2.random(), prog[j][4])
                vals = list(leaves)
                temps = []
                for kind, name, u, v, w in prog:
                    a, b = vals[int(u * len(vals))], vals[int(v * len(vals))]
                    if kind == "u":
                        t = ctx.op(name, a)
                    elif kind == "b":
                        t = ctx.op(name, a, b)
                    elif kind == "s":
                        t = ctx.op("mul", a, ctx.scalar(round(w * 4) / 2))  # 0.0 and 1.0 among the values
                    else:
                        t = ctx.op("add", a, b)
                        ctx.assign(leaves[int(w * 3)], t)
                    temps.append(t)
                    vals.append(t)
                    if w < 0.2 and len(temps) > 2:
                        victim = temps.pop(0)
                        vals = [q for q in vals if q is not victim]
                        ctx.release(victim)
                before = ctx.stats()
                ctx.barrier()
                log.append((delta(ctx, before), ctx.dump_plan(), [(t.shape, ctx.is_materialised(t)) for t in temps]))
                for t in temps:
                    ctx.release(t)
            results[ctx] = log
        assert results[on] == results[off], f"trial {trial}"
        matched += on.stats()["traces_matched"]
        diverged += on.stats()["traces_diverged"]
    assert matched > 100 and diverged > 50, (matched, diverged)  # both paths were exercised


def test_errors_inside_a_matched_trace_are_the_usual_errors():
    on, off = pair()
    out = {}
    for ctx in (on, off):
        x, m = fake(ctx, (16, 16)), fake(ctx, (16, 16), "u8")
        other = lt.LazyContext(device=None)
        foreign = fake(other, (16, 16))
        log = []
        for k in range(5):
            a = ctx.op("exp", x)
            if k == 3:
                for bad in (lambda: ctx.op("add", a, m),            # dtype mismatch
                            lambda: ctx.op("add", a, foreign),      # a handle of another context
                            lambda: ctx.op("row_sum", m)):          # not defined for u8
                    with pytest.raises(lt.LazyTensorError) as err:
                        bad()
                    log.append(err.value.args[0] if err.value.args else str(err.value))
            b = ctx.op("mul", a, a)
            ctx.release(a)
            if k >= 3:
                with pytest.raises(lt.LazyTensorError):
                    ctx.op("neg", a)                                # released: in a matched trace too
            before = ctx.stats()
            ctx.barrier()
            log.append((delta(ctx, before), ctx.dump_plan(), ctx.is_materialised(b)))
            del a, b
        out[ctx] = log
        other.close()
    assert out[on] == out[off]
    assert on.stats()["traces_matched"] >= 1


# ------------------------------------------------------------------ several recording calls in one (lt_op_many)
class _Names:
    pass


def _adam_batch():
    from workloads import traces

    b = lt.Batch()
    p, g, m, v = (b.input() for _ in range(4))
    s = _Names()
    for name in ("beta1", "one_minus_beta1", "beta2", "one_minus_beta2", "sqrt_bc2", "eps", "step_size"):
        setattr(s, name, b.input())
    traces.adam_update(b, p, g, m, v, s)  # the same function that traces on a context builds the batch
    return b


def test_batched_recording_is_the_calls_one_by_one():
    from workloads import traces

    batch = _adam_batch()
    seen = {}
    for mode in ("calls", "batch"):
        ctx = lt.LazyContext(device=None)
        P, G, M, V = ([fake(ctx, (96,)) for _ in range(4)] for _ in range(4))
        log = []
        for step in range(1, 6):
            s = traces.AdamScalars(ctx, step=step)
            for p, g, m, v in zip(P, G, M, V):
                if mode == "calls":
                    traces.adam_update(ctx, p, g, m, v, s)
                else:
                    kept = ctx.record(batch, [p, g, m, v, s.beta1, s.one_minus_beta1, s.beta2, s.one_minus_beta2, s.sqrt_bc2, s.eps, s.step_size])
                    assert kept == []
            if step == 1:
                log.append(ctx.dump_ir())
            before = ctx.stats()
            ctx.barrier()
            log.append((delta(ctx, before), ctx.dump_plan()))
        st = ctx.stats()
        log.append((st["compiles"], st["cache_hits"], st["traces_matched"], st["traces_diverged"]))
        seen[mode] = log
        ctx.close()
    assert seen["calls"] == seen["batch"]
    assert seen["batch"][-1] == (1, 4, 3, 0)


def test_batch_results_errors_and_bad_references():
    ctx = lt.LazyContext(device=None)
    x, y, mask = fake(ctx, (8, 16)), fake(ctx, (8, 16)), fake(ctx, (8, 16), "u8")
    b = lt.Batch()
    a, c_ = b.input(), b.input()
    t = b.op("mul", b.op("add", a, c_), a)
    u = b.op("convert", t, dtype="bf16")
    b.keep(t)
    b.keep(u)
    kept = ctx.record(b, [x, y])
    assert [k.shape for k in kept] == [(8, 16), (8, 16)] and kept[1].dtype == "bf16"
    text = ctx.dump_ir()
    assert text.count("lt::add(") == 1 and text.count("ROOT=") == 2  # the add is a temporary of the batch: no handle, not a root
    ctx.barrier()
    assert ctx.stats()["kernels_launched"] == 1
    # an entry that fails: nothing of the batch is left behind, the error is the failing call's
    bad = lt.Batch()
    p, q = bad.input(), bad.input()
    bad.keep(bad.op("exp", p))
    bad.op("add", p, q)  # f32 + u8
    before = ctx.stats()["nodes_recorded"]
    with pytest.raises(lt.LazyTensorError) as err:
        ctx.record(bad, [x, mask])
    assert "dtype" in str(err.value)
    assert ctx.dump_ir().count("lt::") == 0 and ctx.stats()["nodes_recorded"] == before + 1
    with pytest.raises(ValueError):
        ctx.record(b, [x])
    # operands must name an input or an earlier entry
    import ctypes

    ops = (lt.lt_batch_op * 1)()
    ops[0].opcode, ops[0].n_in, ops[0].in_[0], ops[0].keep = lt.OPCODES["exp"], 1, -1, 1
    res, ins = (ctypes.c_uint64 * 1)(), (ctypes.c_uint64 * 1)(x.handle)
    assert lt._lib.lt_op_many(ctx._ctx, ops, 1, ins, 1, None, res) != 0 and res[0] == 0
    ctx.close()
