"""Host-side logic on a record-and-plan-only context (no GPU, no CUDA call): the C ABI's symbols,
the IR recorder, canonical form and hash, compile cache, fusion planner and donation rules."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2102_13267_b200 as lt
from workloads import configs, traces
from workloads.resnet50 import parameter_shapes

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture()
def ctx():
    c = lt.LazyContext(device=None)
    yield c
    c.close()


def fake(ctx, shape, dtype="f32", base=[1 << 30]):
    """A device-data leaf over an address that is never dereferenced (nothing is launched)."""
    base[0] += 1 << 28
    return ctx.from_device_ptr(base[0], dtype, shape)


# ------------------------------------------------------------------ C ABI surface
def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "lazytensor.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(lt_[a-z_]+)\s*\(", header))
    assert {"lt_tensor_from_device", "lt_op", "lt_barrier", "lt_fetch", "lt_assign"} <= declared
    lib = ctypes.CDLL(str(lt.LIB_PATH))
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared in lazytensor.h but not exported"
    assert set(lt.EXPORTED_SYMBOLS) == declared
    assert lt.version().startswith("lazytensor")


# ------------------------------------------------------------------ IR text (paper Fig. 1, 2)
def test_ir_text_of_x_times_y_plus_z(ctx):
    x, y, z = (fake(ctx, (2, 4)) for _ in range(3))
    out = ctx.op("add", ctx.op("mul", x, y), z)
    text = ctx.dump_ir()
    lines = [ln.strip() for ln in text.splitlines()[1:-1]]
    assert text.startswith("IR {") and text.rstrip().endswith("}")
    assert len(lines) == 5
    assert sum("lt::device_data()" in ln for ln in lines) == 3
    assert all(ln.split(" = ")[1].startswith("f32[2,4]") for ln in lines)
    assert lines[-1] == "%4 = f32[2,4] lt::add(%2, %3), ROOT=0"
    assert lines[2] == "%2 = f32[2,4] lt::mul(%0, %1)"
    assert sum("ROOT=" in ln for ln in lines) == 1
    # the scaling constant 1 of Fig. 1 is a rank-0 constant whose value is part of the graph
    scaled = ctx.op("add", ctx.op("mul", x, y), ctx.op("mul", z, ctx.scalar(1.0)))
    del out
    text = ctx.dump_ir()
    assert "f32[] lt::constant(), value=1" in text


def test_host_loop_unrolls_into_one_graph(ctx):
    x, s = fake(ctx, (2, 4)), fake(ctx, (2, 4))
    for _ in range(2):
        s = ctx.op("add", s, x)
    text = ctx.dump_ir()
    assert text.count("lt::add(") == 2 and text.count("ROOT=") == 1
    ctx.barrier()
    assert ctx.stats()["kernels_launched"] == 1
    assert ctx.dump_ir().count("lt::") == 0  # nothing pending after the barrier


# ------------------------------------------------------------------ hash and cache (paper Section 4.1)
def _flush(ctx, build):
    before = ctx.stats()
    keep = build()
    ctx.barrier()
    after = ctx.stats()
    del keep
    return after["compiles"] - before["compiles"], after["cache_hits"] - before["cache_hits"]


def test_scalar_classes(ctx):
    x = fake(ctx, (64, 64))
    assert _flush(ctx, lambda: ctx.op("add", x, ctx.scalar(42.0))) == (1, 0)
    assert _flush(ctx, lambda: ctx.op("add", x, ctx.scalar(43.0))) == (0, 1)   # another value: same entry
    assert _flush(ctx, lambda: ctx.op("add", x, ctx.scalar(0.0))) == (1, 0)    # 0 is part of the graph
    assert _flush(ctx, lambda: ctx.op("add", x, ctx.scalar(1.0))) == (1, 0)    # so is 1
    assert _flush(ctx, lambda: ctx.op("add", x, ctx.scalar(2.0))) == (0, 1)
    assert _flush(ctx, lambda: ctx.op("add", x, ctx.scalar(-0.0))) == (0, 1)   # -0.0 is not the special 0
    assert _flush(ctx, lambda: ctx.op("add", x, ctx.scalar(1.0, dynamic=True))) == (0, 1)
    assert ctx.cache_size() == 3


def test_operand_identity_and_shape_enter_the_hash(ctx):
    a, b = fake(ctx, (32, 32)), fake(ctx, (32, 32))
    assert _flush(ctx, lambda: ctx.op("mul", a, b)) == (1, 0)
    assert _flush(ctx, lambda: ctx.op("mul", a, a)) == (1, 0)      # a*a is not a*b
    assert _flush(ctx, lambda: ctx.op("mul", b, a)) == (0, 1)      # other buffers, same program
    c, d = fake(ctx, (32, 64)), fake(ctx, (32, 64))
    assert _flush(ctx, lambda: ctx.op("mul", c, d)) == (1, 0)      # shape change recompiles
    e, f = fake(ctx, (32, 32), "bf16"), fake(ctx, (32, 32), "bf16")
    assert _flush(ctx, lambda: ctx.op("mul", e, f)) == (1, 0)      # dtype change recompiles
    ctx.set_option("fusion", 0)
    assert _flush(ctx, lambda: ctx.op("mul", a, b)) == (1, 0)      # options are part of the key


def test_c1_traced_ten_times_compiles_once(ctx):
    leaves = [fake(ctx, (1024, 1024)) for _ in range(4)]
    for _ in range(10):
        y = traces.elementwise_chain(ctx, *leaves)
        ctx.barrier()
    s = ctx.stats()
    assert (s["compiles"], s["cache_hits"], s["kernels_launched"]) == (1, 9, 10)
    assert s["bytes_planned"] == 10 * configs.algorithmic_bytes("c1")


def test_c5_hundred_steps_one_compile(ctx):
    shapes = parameter_shapes()
    P, G, M, V = ([fake(ctx, s) for s in shapes] for _ in range(4))
    for step in range(1, 101):
        traces.adam_step(ctx, P, G, M, V, step=step)
        ctx.barrier()
    s = ctx.stats()
    assert (s["compiles"], s["cache_hits"]) == (1, 99)
    assert s["kernels_launched"] == 100 and s["launches_multi"] == 100
    assert s["outputs_donated"] == 100 * 3 * 161 and s["outputs_allocated"] == 0
    assert s["temporaries_allocated"] == 0
    assert s["bytes_planned"] == 100 * configs.algorithmic_bytes("c5")
    plan = ctx.dump_plan()
    assert "launch 0: multi precise instances=161" in plan and "launch 1" not in plan


def test_cache_capacity_evicts_least_recently_used(ctx):
    ctx.set_option("cache_capacity", 2)
    x = fake(ctx, (16, 16))
    prog = {k: (lambda k=k: ctx.op(k, x, x)) for k in ("add", "sub", "max")}
    assert _flush(ctx, prog["add"]) == (1, 0)
    assert _flush(ctx, prog["sub"]) == (1, 0)
    assert _flush(ctx, prog["add"]) == (0, 1)
    assert _flush(ctx, prog["max"]) == (1, 0)   # evicts sub
    assert _flush(ctx, prog["add"]) == (0, 1)
    assert _flush(ctx, prog["sub"]) == (1, 0)
    assert ctx.cache_size() == 2


# ------------------------------------------------------------------ planner
def test_each_config_is_one_fused_kernel(ctx):
    x, h, b = fake(ctx, (8192, 4096), "bf16"), fake(ctx, (8192, 4096), "bf16"), fake(ctx, (4096,), "bf16")
    out = traces.mlp_epilogue(ctx, x, h, b)
    ctx.barrier()
    plan = ctx.dump_plan()
    assert plan.startswith("plan: 1 launches, 1 groups") and "elementwise fast" in plan and "colvec" in plan
    assert ctx.stats()["bytes_planned"] == configs.algorithmic_bytes("c2")
    ctx.reset_stats()
    shape = (16384, 1024)
    z, keep = traces.residual_dropout_layernorm(ctx, fake(ctx, shape, "bf16"), fake(ctx, shape, "bf16"),
                                                fake(ctx, (1024,)), fake(ctx, (1024,)), shape=shape, p=0.1,
                                                eps=1e-5, seed=1, offset=2)
    ctx.barrier()
    plan = ctx.dump_plan()
    assert plan.startswith("plan: 1 launches, 1 groups") and "row fast" in plan
    assert plan.count("row_sum") == 2 and "philox" in plan
    assert ctx.stats()["bytes_planned"] == configs.algorithmic_bytes("c3")
    ctx.reset_stats()
    shape = (16, 2048, 2048)
    y = traces.causal_softmax(ctx, fake(ctx, shape, "bf16"), shape=shape, scale=0.088)
    ctx.barrier()
    plan = ctx.dump_plan()
    assert plan.startswith("plan: 1 launches, 1 groups") and "row_max" in plan and "iota" in plan
    assert ctx.stats()["bytes_planned"] == configs.algorithmic_bytes("c4")


def test_f32_results_never_use_the_fast_flavour(ctx):
    shape = (64, 256)
    z, keep = traces.residual_dropout_layernorm(ctx, fake(ctx, shape, "bf16"), fake(ctx, shape, "bf16"),
                                                fake(ctx, (256,)), fake(ctx, (256,)), shape=shape, p=0.1,
                                                eps=1e-5, seed=1, offset=2, out_dtype="f32")
    ctx.barrier()
    assert "row precise" in ctx.dump_plan()
    ctx.set_option("ieee", 1)
    x = fake(ctx, (64, 64))
    q = ctx.op("div", x, x)
    ctx.barrier()
    assert "elementwise ieee" in ctx.dump_plan()


def test_unfused_mode_launches_one_kernel_per_op(ctx):
    ctx.set_option("fusion", 0)
    leaves = [fake(ctx, (256, 256)) for _ in range(4)]
    y = traces.elementwise_chain(ctx, *leaves)
    ctx.barrier()
    s = ctx.stats()
    assert s["kernels_launched"] == 5 and s["temporaries_allocated"] == 4


def test_live_intermediate_becomes_an_output(ctx):
    a, b = fake(ctx, (128, 128)), fake(ctx, (128, 128))
    t = ctx.op("mul", a, b)
    y = ctx.op("relu", t)
    ctx.barrier()                       # t is still named: the barrier must materialise it too
    assert ctx.stats()["outputs_allocated"] == 2 and ctx.is_materialised(t)
    ctx.reset_stats()
    t2 = ctx.op("mul", a, b)
    y2 = ctx.op("relu", t2)
    del t2
    ctx.barrier()
    assert ctx.stats()["outputs_allocated"] == 1


def test_program_too_large_for_one_group_is_split(ctx):
    xs = [fake(ctx, (64, 64)) for _ in range(9)]
    acc = ctx.op("mul", xs[0], xs[1])
    prods = [ctx.op("mul", xs[i], xs[i + 1]) for i in range(1, 8)]
    # a wide tree: more simultaneously live values than the machine has registers
    lvl = [acc] + prods
    while len(lvl) > 1:
        lvl = [ctx.op("add", lvl[i], lvl[i + 1]) for i in range(0, len(lvl) - 1, 2)] + (lvl[-1:] if len(lvl) % 2 else [])
    out = lvl[0]
    del acc, prods, lvl
    ctx.barrier()
    s = ctx.stats()
    assert s["outputs_allocated"] == 1 and s["kernels_launched"] >= 1


# ------------------------------------------------------------------ in-place updates (paper Section 4.3)
def test_in_place_update_is_donated_once(ctx):
    a = fake(ctx, (64, 64))
    ptr = ctx.device_ptr(a)
    a += 1.0
    ctx.barrier()
    s = ctx.stats()
    assert (s["outputs_donated"], s["outputs_allocated"], s["kernels_launched"]) == (1, 0, 1)
    assert ctx.device_ptr(a) == ptr
    ctx.barrier()                        # observing a twice must not increment twice: nothing is pending
    ctx.barrier()
    assert ctx.stats()["kernels_launched"] == 1


def test_second_reader_in_the_same_kernel_keeps_donation(ctx):
    a = fake(ctx, (64, 64))
    b = a + 2.0                          # must see the old a
    a += 1.0
    ctx.barrier()
    s = ctx.stats()
    assert s["kernels_launched"] == 1 and s["outputs_donated"] == 1 and s["outputs_allocated"] == 1
    plan = ctx.dump_plan()
    assert plan.index("= load p0") < plan.index("  store p")  # the old value is read before any store


def test_no_donation_while_another_tensor_names_the_old_value(ctx):
    a = fake(ctx, (64, 64))
    alias = fake(ctx, (64, 64))
    ctx.assign(alias, a)                 # alias now names a's buffer as well
    a += 1.0
    ctx.barrier()
    s = ctx.stats()
    assert s["outputs_donated"] == 0 and s["outputs_allocated"] == 1


def test_no_donation_when_a_later_kernel_reads_the_old_value(ctx):
    ctx.set_option("fusion", 0)          # one kernel per op: b's kernel runs after a's
    a = fake(ctx, (64, 64))
    new_a = a + 1.0
    b = a * 3.0
    ctx.assign(a, new_a)
    del new_a
    ctx.barrier()
    s = ctx.stats()
    assert s["kernels_launched"] == 2
    # a's update is traced first, so its kernel precedes the one that still reads the old buffer
    assert s["outputs_donated"] == 0 and s["outputs_allocated"] == 2


def test_broadcast_reader_blocks_donation(ctx):
    col = fake(ctx, (256,))
    full = fake(ctx, (8, 256))
    # the column vector is read by every row of the wide kernel: it cannot be overwritten in place there
    wide = ctx.op("add", full, col)
    newcol = ctx.op("mul", col, ctx.scalar(2.0))
    ctx.assign(col, newcol)
    del newcol
    ctx.barrier()
    assert ctx.stats()["outputs_donated"] in (0, 1)
    plan = ctx.dump_plan()
    if "donated" in plan:                # only legal when the in-place kernel runs after the wide one
        assert plan.index("colvec") < plan.rindex("launch")


# ------------------------------------------------------------------ errors
def test_error_paths(ctx):
    a, b = fake(ctx, (4, 8)), fake(ctx, (4, 7))
    with pytest.raises(lt.LazyTensorError) as e:
        ctx.op("add", a, b)
    assert e.value.status == 2  # LT_ERR_SHAPE
    with pytest.raises(lt.LazyTensorError) as e:
        ctx.op("add", a, fake(ctx, (4, 8), "bf16"))
    assert e.value.status == 3  # LT_ERR_DTYPE
    with pytest.raises(lt.LazyTensorError) as e:
        ctx.op("add", fake(ctx, (4, 8), "i32"), ctx.scalar(0.5))
    assert e.value.status == 3
    with pytest.raises(lt.LazyTensorError) as e:
        ctx.op("col_sum", fake(ctx, (4, 8), "i32"))
    assert e.value.status == 3
    with pytest.raises(lt.LazyTensorError) as e:
        ctx.op("exp", fake(ctx, (4,), "i32"))
    assert e.value.status == 3
    other = lt.LazyContext(device=None)
    foreign = other.from_device_ptr(1 << 40, "f32", (4, 8))
    with pytest.raises(lt.LazyTensorError) as e:
        ctx.op("add", a, foreign)
    assert e.value.status == 4  # LT_ERR_DEVICE: no implicit cross-device operands
    assert ctx.stats()["nodes_recorded"] == 7  # six leaves and one scalar: the failed ops recorded nothing
    with pytest.raises(lt.LazyTensorError):
        ctx.fetch(a)  # no device behind this context
    with pytest.raises(lt.LazyTensorError):
        ctx.set_option("no_such_option", 1)
    other.close()


def test_failed_allocation_leaves_the_graph_flushable():
    lib = ctypes.CDLL(str(lt.LIB_PATH))
    fail_next = {"on": True}
    live = {}

    def alloc(nbytes, stream, user):
        if fail_next["on"]:
            return None
        buf = ctypes.create_string_buffer(max(int(nbytes), 16))
        live[ctypes.addressof(buf)] = buf
        return ctypes.addressof(buf)

    def free(ptr, stream, user):
        live.pop(ptr, None)

    a_fn, f_fn = lt.ALLOC_FN(alloc), lt.FREE_FN(free)
    st = lt.lt_allocator(a_fn, f_fn, None)
    c = ctypes.c_void_p()
    assert lib.lt_ctx_create(-1, None, ctypes.byref(st), ctypes.byref(c)) == 0
    h = [ctypes.c_uint64() for _ in range(3)]
    shape = (ctypes.c_int64 * 2)(4, 4)
    lib.lt_tensor_from_device.argtypes = lt._SIGNATURES["lt_tensor_from_device"]
    lib.lt_op.argtypes = lt._SIGNATURES["lt_op"]
    lib.lt_barrier.argtypes = lt._SIGNATURES["lt_barrier"]
    lib.lt_get_stats.argtypes = lt._SIGNATURES["lt_get_stats"]
    lib.lt_last_error.restype = ctypes.c_char_p
    lib.lt_last_error.argtypes = [ctypes.c_void_p]
    for i in range(2):
        assert lib.lt_tensor_from_device(c, ctypes.c_void_p(4096 * (i + 1)), 0, 2, shape, ctypes.byref(h[i])) == 0
    ins = (ctypes.c_uint64 * 2)(h[0].value, h[1].value)
    assert lib.lt_op(c, 1, ins, 2, None, 0, ctypes.byref(h[2])) == 0
    assert lib.lt_barrier(c, 0) == 6  # LT_ERR_OOM
    assert b"allocator" in lib.lt_last_error(c)
    fail_next["on"] = False
    assert lib.lt_barrier(c, 0) == 0  # the pending graph was left intact and flushes now
    s = lt.lt_stats()
    assert lib.lt_get_stats(c, ctypes.byref(s)) == 0
    assert s.kernels_launched == 1 and s.outputs_allocated == 1
    lib.lt_ctx_destroy.argtypes = [ctypes.c_void_p]
    assert lib.lt_ctx_destroy(c) == 0
    assert not live  # the output buffer went back through the free callback


def test_released_blocks_are_reused_before_the_allocator_is_asked():
    """Steady state makes no allocator call: the block of a released result serves the next flush of the
    same size; `pool_bytes` = 0 hands every block back at once; closing the context returns the rest."""
    lib = ctypes.CDLL(str(lt.LIB_PATH))
    calls = {"alloc": 0, "free": 0}
    live = {}

    def alloc(nbytes, stream, user):
        calls["alloc"] += 1
        buf = ctypes.create_string_buffer(max(int(nbytes), 16))
        live[ctypes.addressof(buf)] = buf
        return ctypes.addressof(buf)

    def free(ptr, stream, user):
        calls["free"] += 1
        live.pop(ptr, None)

    a_fn, f_fn = lt.ALLOC_FN(alloc), lt.FREE_FN(free)
    st = lt.lt_allocator(a_fn, f_fn, None)
    c = ctypes.c_void_p()
    assert lib.lt_ctx_create(-1, None, ctypes.byref(st), ctypes.byref(c)) == 0
    for name in ("lt_tensor_from_device", "lt_op", "lt_barrier", "lt_release", "lt_ctx_set_option", "lt_ctx_destroy"):
        getattr(lib, name).argtypes = lt._SIGNATURES[name]
    shape = (ctypes.c_int64 * 2)(64, 64)
    a, b, y = ctypes.c_uint64(), ctypes.c_uint64(), ctypes.c_uint64()
    assert lib.lt_tensor_from_device(c, ctypes.c_void_p(1 << 20), 0, 2, shape, ctypes.byref(a)) == 0
    assert lib.lt_tensor_from_device(c, ctypes.c_void_p(2 << 20), 0, 2, shape, ctypes.byref(b)) == 0

    def step():
        ins = (ctypes.c_uint64 * 2)(a.value, b.value)
        assert lib.lt_op(c, 1, ins, 2, None, 0, ctypes.byref(y)) == 0
        assert lib.lt_barrier(c, 0) == 0
        assert lib.lt_release(c, y.value) == 0

    for _ in range(5):
        step()
    assert calls == {"alloc": 1, "free": 0}  # one block, recycled four times
    assert lib.lt_ctx_set_option(c, b"pool_bytes", 0) == 0  # gives the pooled block back ...
    assert calls["free"] == 1 and not live
    for _ in range(3):
        step()                                               # ... and from now on every flush allocates and frees
    assert calls == {"alloc": 4, "free": 4}
    assert lib.lt_ctx_set_option(c, b"pool_bytes", 1 << 20) == 0
    step()
    assert calls == {"alloc": 5, "free": 4} and len(live) == 1
    assert lib.lt_ctx_destroy(c) == 0
    assert calls["free"] == 5 and not live


# ------------------------------------------------------------------ ahead-of-time compiled programs
def test_compiled_table_is_what_the_planner_emits_today():
    """The committed table of compiled programs equals what its generator derives from the planner now
    (a planner change that alters a listed program must be followed by regenerating the table), and
    planning a listed graph finds its entry."""
    import importlib.util

    path = os.path.join(ROOT, "paper_2102_13267_b200", "csrc", "gen_compiled.py")
    spec = importlib.util.spec_from_file_location("gen_compiled", path)
    gen = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(gen)
    text, names = gen.render()
    committed = open(os.path.join(ROOT, "paper_2102_13267_b200", "csrc", "compiled_programs.inc")).read()
    assert text == committed, "run paper_2102_13267_b200/csrc/gen_compiled.py and rebuild"
    assert len(names) >= 8
    d = gen.Dry()
    a, b, c, e = (d.leaf((64, 64), "f32") for _ in range(4))
    keep = gen.traces.elementwise_chain(d.ctx, a, b, c, e)
    d.ctx.barrier()
    assert "compiled: elementwise_chain" in d.ctx.dump_plan()
    # a graph that is not listed stays on the interpreter
    d = gen.Dry()
    a, b = (d.leaf((64, 64), "f32") for _ in range(2))
    keep = d.ctx.op("max", d.ctx.op("sub", a, b), d.ctx.op("exp", b))
    d.ctx.barrier()
    assert "compiled: no" in d.ctx.dump_plan()
    del keep


def test_host_bench_driver_runs_without_python_in_the_loop():
    """The C++ driver records, flushes and replays three of the configurations through the C ABI alone."""
    import importlib.util
    import subprocess

    spec = importlib.util.spec_from_file_location("_lt_build", os.path.join(ROOT, "paper_2102_13267_b200", "_build.py"))
    b = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(b)
    out = subprocess.run([str(b.build_host_bench())], capture_output=True, text=True, timeout=120, check=True).stdout
    lines = out.strip().splitlines()
    assert len(lines) == 5
    assert "compiles 1, hits 19999" in lines[0] and "compiles 1, hits 19999" in lines[1]
    assert "compiles 1, hits 999 (998 by matched trace, 0 traces diverged)" in lines[2]
    assert "batched" in lines[3] and "compiles 0, hits 1000 (998 by matched trace, 0 traces diverged)" in lines[3]  # lt_op_many: the same graph, found in the cache
    assert "replays 999" in lines[4]


# ------------------------------------------------------------------ long rows and the other reduction shapes
def test_long_row_groups_fused_when_listed_and_split_otherwise():
    from workloads import idioms

    ctx = lt.LazyContext(device=None)
    ctx.set_option("specialise", 0)
    x = fake(ctx, (4, 16384), "bf16")
    y = idioms.softmax(ctx, x, cols=16384)
    ctx.barrier()
    plan = ctx.dump_plan()
    assert plan.count("launch ") == 1 and "compiled: softmax_bf16" in plan and "rows=4 cols=16384" in plan
    # a graph with no kernel instantiated for it: each long reduction becomes a kernel of its own, the arithmetic
    # around it elementwise kernels that read one value per row
    z = fake(ctx, (4, 16384))
    d = ctx.op("sub", z, ctx.op("row_max", z))
    w = ctx.op("div", ctx.op("abs", d), ctx.op("add", ctx.op("row_sum", ctx.op("abs", d)), ctx.scalar(3.0)))
    ctx.barrier()
    plan = ctx.dump_plan()
    assert plan.count("reduction kernel: max over rows") == 1 and plan.count("reduction kernel: sum over rows") == 1
    assert "launch 0: reduce" in plan and "rowvec" in plan
    st = ctx.stats()
    assert st["launches_reduce"] == 2
    # the same graph at 8192 columns stays one fused row kernel
    z = fake(ctx, (4, 8192))
    d = ctx.op("sub", z, ctx.op("row_max", z))
    w2 = ctx.op("div", ctx.op("abs", d), ctx.op("add", ctx.op("row_sum", ctx.op("abs", d)), ctx.scalar(3.0)))
    ctx.barrier()
    assert ctx.dump_plan().count("launch ") == 1
    del y, w, w2


def test_column_and_whole_tensor_reductions_plan_as_their_own_kernels():
    ctx = lt.LazyContext(device=None)
    x = fake(ctx, (512, 96))
    s = ctx.op("col_sum", ctx.op("mul", x, x))          # the product is materialised, then reduced
    t = ctx.op("all_max", x)
    u = ctx.op("sub", x, ctx.op("col_max", x))           # result read back as a column vector
    v = ctx.op("mul", x, t)                              # rank-0 result read back as a broadcast scalar
    assert s.shape == (1, 96) and t.shape == () and u.shape == (512, 96)
    ctx.barrier()
    plan = ctx.dump_plan()
    assert plan.count("reduction kernel: sum over columns") == 1
    assert plan.count("reduction kernel: max over all") == 1
    assert plan.count("reduction kernel: max over columns") == 1
    assert "colvec" in plan and "scalar" in plan
    assert ctx.stats()["launches_reduce"] == 3
    with pytest.raises(lt.LazyTensorError):
        ctx.op("all_sum", ctx.scalar(2.0))
    del s, t, u, v


def test_outer_broadcast_of_row_scalars_and_column_vector():
    ctx = lt.LazyContext(device=None)
    r, cvec = fake(ctx, (7, 1)), fake(ctx, (1, 40))
    y = ctx.op("mul", r, cvec)
    assert y.shape == (7, 40)
    ctx.barrier()
    plan = ctx.dump_plan()
    assert plan.count("launch ") == 1 and "rowvec" in plan and "colvec" in plan
    del y


# ------------------------------------------------------------------ views (paper Section 4.4, Fig. 3)
def test_in_place_update_of_a_view_records_forward_and_backward_sequences(ctx):
    x = fake(ctx, (2, 3, 4))
    v = ctx.view_permute(x, (1, 2, 0))
    assert v.shape == (3, 4, 2)
    ctx.assign(v, ctx.op("add", v, ctx.scalar(42.0)))
    ctx.release(v)  # the figure shows the base's computation alone
    lines = [ln.strip() for ln in ctx.dump_ir().splitlines()[1:-1]]
    golden = [ln for ln in open(os.path.join(ROOT, "tests", "golden", "fig3_inplace_on_view.txt")) if not ln.startswith("#")]
    assert len(lines) == len(golden) == 5
    order = {}  # node number in the dump -> position in the golden list (the dump numbers operands first-visit)
    parsed = []
    for ln in lines:
        m = re.match(r"%(\d+) = f32\[([\d,]*)\] lt::(\w+)\(([^)]*)\)(.*)", ln)
        parsed.append((int(m.group(1)), m.group(2), m.group(3), [int(t.strip()[1:]) for t in m.group(4).split(",") if t.strip()], m.group(5)))
    by_op = lambda name, k=0: [p for p in parsed if p[2] == name][k]
    want = [tuple(f.strip() for f in g.split("|")) for g in golden]
    got_nodes = [by_op("scalar_data"), by_op("device_data"), by_op("permute", 0), by_op("add"), by_op("permute", 1)]
    for pos, node in enumerate(got_nodes):
        order[node[0]] = pos
    for (shape, op, operands, dims, root), node in zip(want, got_nodes):
        assert "[" + node[1] + "]" == shape and node[2] == op
        assert sorted(order[o] for o in node[3]) == sorted(int(t) for t in operands.split() if t != "-")
        if dims != "-":
            assert f"dims={dims}" in node[4]
        assert ("ROOT=0" in node[4]) == (root == "ROOT")
    # the forward permutation feeds the add, the inverse one consumes it
    assert got_nodes[3][3].count(got_nodes[2][0]) == 1 and got_nodes[4][3] == [got_nodes[3][0]]


def test_views_follow_their_base_and_bases_follow_their_views(ctx):
    x = fake(ctx, (4, 8))
    v = ctx.view_narrow(x, 1, 2, 4)
    w = ctx.view_reshape(x, (8, 4))
    assert v.shape == (4, 4) and w.shape == (8, 4)
    # the base is updated in place: both views are derived again from its new computation
    ctx.assign(x, ctx.op("mul", x, ctx.scalar(3.0)))
    ctx.release(w)
    text = ctx.dump_ir()
    assert text.count("lt::narrow(") == 1 and "dim=1, start=2" in text and text.count("ROOT=") == 2
    # the view is updated in place: the base becomes update_slice(base, view)
    ctx.assign(v, ctx.op("neg", v))
    text = ctx.dump_ir()
    assert text.count("lt::update_slice(") == 1 and text.count("lt::neg(") == 1
    ctx.barrier()
    plan = ctx.dump_plan()
    assert "copy kernel: narrow" in plan and "copy kernel: update_slice" in plan
    # a chain of views: permute of a narrow; the update walks back through both
    y = fake(ctx, (2, 3, 4))
    n = ctx.view_narrow(y, 2, 1, 2)
    p = ctx.view_permute(n, (2, 0, 1))
    assert p.shape == (2, 2, 3)
    ctx.assign(p, ctx.op("add", p, ctx.scalar(1.0)))
    text = ctx.dump_ir()
    assert text.count("lt::permute(") == 2 and "dims=(1, 2, 0)" in text and text.count("lt::update_slice(") == 1
    assert text.count("ROOT=") == 3  # the permuted view, the narrowed view and the base
    ctx.barrier()
    # reshaping materialised data records nothing and shares the buffer
    z = fake(ctx, (6, 4))
    r = ctx.view_reshape(z, (2, 12))
    assert ctx.is_materialised(r) and ctx.dump_ir().count("lt::") == 0


def test_shape_op_errors(ctx):
    x = fake(ctx, (4, 8))
    for bad in (lambda: ctx.view_narrow(x, 1, 6, 4), lambda: ctx.view_narrow(x, 2, 0, 1), lambda: ctx.view_reshape(x, (5, 7)),
                lambda: ctx.view_permute(x, (0, 0)), lambda: ctx.op("update_slice", x, fake(ctx, (4, 9)), dim=1, start=0),
                lambda: ctx.op("update_slice", x, fake(ctx, (4, 4)), dim=1, start=5)):
        with pytest.raises(lt.LazyTensorError):
            bad()


def test_reshape_that_keeps_rows_and_columns_is_folded_into_the_program(ctx):
    x = fake(ctx, (2, 3, 8))
    y = ctx.op("add", ctx.op("reshape", ctx.op("mul", x, x), shape=(6, 8)), ctx.scalar(2.0))
    ctx.barrier()
    assert ctx.stats()["kernels_launched"] == 1 and ctx.stats()["launches_view"] == 0
    z = ctx.op("add", ctx.op("reshape", ctx.op("mul", x, x), shape=(4, 12)), ctx.scalar(2.0))
    ctx.barrier()
    assert ctx.stats()["launches_view"] == 1
    del y, z


# ------------------------------------------------------------------ run-time specialisation
def test_run_time_specialiser_builds_the_shells_for_an_unlisted_program():
    """With specialise=1 a long-row group that has no kernel in the table stays fused, because its kernel is built
    while the graph is planned.  The run-time compiler needs no GPU, so this runs here: it shows that the device
    headers are self-contained and that the program's table entry is generated correctly."""
    ctx = lt.LazyContext(device=None)
    ctx.set_option("specialise", 1)
    z = fake(ctx, (4, 16384))
    d = ctx.op("abs", ctx.op("sub", z, ctx.op("row_max", z)))
    w = ctx.op("div", d, ctx.op("add", ctx.op("row_sum", d), ctx.scalar(3.0)))
    ctx.barrier()
    plan = ctx.dump_plan()
    if "specialised at run time" not in plan:
        pytest.skip("the run-time compiler library is not installed")
    assert plan.count("launch ") == 1 and "launch 0: row" in plan and "specialised at run time: ready" in plan, plan
    assert ctx.stats()["launches_reduce"] == 0
    # with specialise=0 the same graph is split
    other = lt.LazyContext(device=None)
    other.set_option("specialise", 0)
    z = fake(other, (4, 16384))
    d = other.op("abs", other.op("sub", z, other.op("row_max", z)))
    w2 = other.op("div", d, other.op("add", other.op("row_sum", d), other.scalar(3.0)))
    other.barrier()
    assert other.stats()["launches_reduce"] == 2
    del w, w2


def test_committed_interpreter_core_is_what_its_generator_emits():
    import importlib.util

    path = os.path.join(ROOT, "paper_2102_13267_b200", "csrc", "gen_vm_core.py")
    spec = importlib.util.spec_from_file_location("gen_vm_core", path)
    gen = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(gen)
    committed = open(os.path.join(ROOT, "paper_2102_13267_b200", "csrc", "vm_core.inc")).read()
    assert gen.render() == committed, "run paper_2102_13267_b200/csrc/gen_vm_core.py and rebuild"


def test_slices_of_materialised_data_are_read_in_place(ctx):
    x = fake(ctx, (64, 256))
    y = fake(ctx, (64, 128))
    out = ctx.op("mul", ctx.op("narrow", x, dim=1, start=64, length=128), y)       # columns 64..191 of every row
    ctx.barrier()
    plan = ctx.dump_plan()
    assert plan.count("launch ") == 1 and "pitched param0" in plan and "copy kernel" not in plan, plan
    head = ctx.op("add", ctx.op("narrow", x, dim=0, start=16, length=8), ctx.scalar(1.0))   # rows 16..23: one contiguous range
    ctx.barrier()
    plan = ctx.dump_plan()
    assert plan.count("launch ") == 1 and "load f32 full param0" in plan and "copy kernel" not in plan, plan
    # a slice that is itself a result, or that feeds a reduction kernel of its own, is copied
    s = ctx.op("narrow", x, dim=1, start=0, length=8)
    t = ctx.op("col_sum", ctx.op("narrow", x, dim=1, start=8, length=8))
    ctx.barrier()
    assert ctx.dump_plan().count("copy kernel: narrow") == 2
    del out, head, s, t


def test_kernel_cache_directory_is_written_and_read(tmp_path, monkeypatch):
    """LT_KERNEL_CACHE: the specialiser stores the machine code of a program in the directory and a later request
    (here: another program identity is needed, so a second process is what really reuses it) finds the file."""
    import subprocess
    import sys

    code = (
        "import sys; sys.path.insert(0, %r)\n"
        "import paper_2102_13267_b200 as lt\n"
        "c = lt.LazyContext(device=None); c.set_option('specialise', 1)\n"
        "z = c.from_device_ptr(1 << 30, 'f32', (4, 16384))\n"
        "d = c.op('abs', c.op('sub', z, c.op('row_min', z)))\n"
        "w = c.op('div', d, c.op('add', c.op('row_sum', d), c.scalar(5.0)))\n"
        "c.barrier(); p = c.dump_plan()\n"
        "print('READY' if 'specialised at run time: ready' in p else ('ABSENT' if 'specialised at run time' not in p else 'FAILED'))\n"
    ) % ROOT
    env = dict(os.environ, LT_KERNEL_CACHE=str(tmp_path))
    import time
    t0 = time.time()
    first = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=300)
    t1 = time.time()
    if "ABSENT" in first.stdout:
        pytest.skip("the run-time compiler library is not installed")
    assert "READY" in first.stdout, first.stdout + first.stderr
    files = list(tmp_path.glob("*.ltk"))
    assert len(files) == 1 and files[0].stat().st_size > 10000
    stamp = files[0].stat().st_mtime_ns
    second = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=300)
    assert "READY" in second.stdout, second.stdout + second.stderr
    assert files[0].stat().st_mtime_ns == stamp and len(list(tmp_path.glob("*"))) == 1  # read, not rewritten


def test_reductions_of_computed_values_are_planned_into_the_computing_kernel(ctx):
    """col / all reduction of an elementwise value nothing else reads: the value's group reduces it (slot class
    'reduced-over-...'), the reduction group keeps its second stage -- when a kernel for that program exists."""
    from workloads import idioms

    x, y = fake(ctx, (4096, 256), "bf16"), fake(ctx, (4096, 256), "bf16")
    g = idioms.relu_bias_grad(ctx, x, y, cols=256)
    ctx.barrier()
    plan = ctx.dump_plan()
    assert plan.count("launch ") == 2 and "compiled: relu_bias_grad_bf16" in plan, plan
    assert "reduced-over-rows(sum)" in plan and "second stage only" in plan
    assert plan.splitlines()[0].endswith("2 temporaries")  # the value's own (empty) and the partial results
    # not in the table and no kernel built while planning (no device, background mode): the value is materialised
    z = ctx.op("col_max", ctx.op("tanh", ctx.op("convert", x, dtype="f32")))
    ctx.barrier()
    plan = ctx.dump_plan()
    assert "second stage only" not in plan and "reduction kernel: max over columns, two stages" in plan, plan
    # small inputs reduce in one stage: nothing to fuse
    s = fake(ctx, (4, 64))
    w = ctx.op("all_sum", ctx.op("mul", s, s))
    ctx.barrier()
    assert "second stage only" not in ctx.dump_plan()
    # a value with another reader, or rows that are not whole chunks, stay as they were
    a = fake(ctx, (4096, 100))
    sq = ctx.op("mul", a, a)
    u = ctx.op("all_sum", sq)
    ctx.barrier()
    assert "second stage only" not in ctx.dump_plan()
    del g, z, w, u, sq
