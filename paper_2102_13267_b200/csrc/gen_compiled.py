#!/usr/bin/env python
"""Generates compiled_programs.inc: the register programs that get an ahead-of-time compiled kernel.

Each entry is the program the planner emits for one traced graph (instructions, prologue length,
slot dtypes and classes, kernel family, arithmetic flavour), taken from the `key:` line of the plan
dump of a record-and-plan-only context.  Shapes, pointers and immediates are not part of an entry:
one entry serves every extent and every value of the run-time scalars.  To give another graph a
compiled kernel, add its trace to `programs()` and rerun:

    python paper_2102_13267_b200/csrc/gen_compiled.py

The library must already be built (any table will do; the planner does not depend on it), and is
rebuilt afterwards by the usual build step.  The output is committed.
"""
from __future__ import annotations

import math
import sys
from pathlib import Path

HERE = Path(__file__).resolve().parent
sys.path.insert(0, str(HERE.parent.parent))

import paper_2102_13267_b200 as lt  # noqa: E402
from workloads import idioms, traces  # noqa: E402

NT = 3          # LT_VM_NT
OP_MOV_T_ACC = 1
OP_ST = 20
OP_LD = 51      # +d, d < NT: temporary, d == NT: ACC


class Dry:
    """A record-and-plan-only context with inputs over addresses that are never dereferenced."""

    def __init__(self, **options):
        self.ctx = lt.LazyContext(device=None)
        for k, v in options.items():
            self.ctx.set_option(k, v)
        self.base = 1 << 30

    def leaf(self, shape, dtype):
        self.base += 1 << 28
        return self.ctx.from_device_ptr(self.base, dtype, shape)

    def keys(self):
        self.ctx.barrier()
        return [ln.strip()[5:] for ln in self.ctx.dump_plan().splitlines() if ln.strip().startswith("key: ")]


def programs():
    """(name, keys) of every graph that gets compiled kernels."""
    out = []
    d = Dry()
    a, b, c, e = (d.leaf((64, 64), "f32") for _ in range(4))
    keep = traces.elementwise_chain(d.ctx, a, b, c, e)
    out.append(("elementwise_chain", d.keys()))
    for prim in (False, True):
        d = Dry()
        x, h = (d.leaf((16, 64), "bf16") for _ in range(2))
        keep = traces.mlp_epilogue(d.ctx, x, h, d.leaf((64,), "bf16"), primitive_gelu=prim)
        out.append(("mlp_epilogue_primitive" if prim else "mlp_epilogue", d.keys()))
    for od in ("bf16", "f32"):
        d = Dry()
        x, h = (d.leaf((16, 64), "bf16") for _ in range(2))
        g, be = (d.leaf((64,), "f32") for _ in range(2))
        keep = traces.residual_dropout_layernorm(d.ctx, x, h, g, be, shape=(16, 64), p=0.1, eps=1e-5, seed=1, offset=0, out_dtype=od)
        out.append((f"residual_dropout_layernorm_{od}", d.keys()))
    # the same normalisation without dropout (evaluation mode)
    d = Dry()
    x, h = (d.leaf((16, 64), "bf16") for _ in range(2))
    g, be = (d.leaf((64,), "f32") for _ in range(2))
    keep = traces.residual_layernorm(d.ctx, x, h, g, be, shape=(16, 64), eps=1e-5)
    out.append(("residual_layernorm_bf16", d.keys()))
    for od in ("bf16", "f32"):
        d = Dry()
        keep = traces.causal_softmax(d.ctx, d.leaf((2, 64, 64), "bf16"), shape=(2, 64, 64), scale=1 / math.sqrt(128), out_dtype=od)
        out.append((f"causal_softmax_{od}", d.keys()))
    # Adam with the default arithmetic (division and square root within 2 ulp) and with ieee=1 (correctly rounded:
    # bit-identical to an op-by-op binary32 evaluation)
    for opts, suffix in (({}, ""), ({"ieee": 1}, "_ieee")):
        d = Dry(**opts)
        shapes = [(64,), (128,)]
        P, G, M, V = ([d.leaf(s, "f32") for s in shapes] for _ in range(4))
        traces.adam_step(d.ctx, P, G, M, V, step=1)
        out.append(("adam_step" + suffix, d.keys()))
    # the data-parallel step: the summed gradient is scaled by a run-time 1 / world size inside the same program
    d = Dry()
    shapes = [(64,), (128,)]
    P, G, M, V = ([d.leaf(s, "f32") for s in shapes] for _ in range(4))
    sc = traces.AdamScalars(d.ctx, step=1)
    inv = d.ctx.scalar(0.5, dynamic=True)
    for p_, g_, m_, v_ in zip(P, G, M, V):
        traces.adam_update(d.ctx, p_, d.ctx.op("mul", g_, inv), m_, v_, sc)
    out.append(("adam_step_data_parallel", d.keys()))
    d = Dry(ieee=1)
    a, b, c, e = (d.leaf((64, 64), "f32") for _ in range(4))
    keep = traces.elementwise_chain(d.ctx, a, b, c, e)
    out.append(("elementwise_chain_ieee", d.keys()))
    # common fusion groups beyond the benchmark's (workloads/idioms.py)
    for name, kinds, trace in idioms.ALL:
        d = Dry()
        ins = [d.leaf((16, 64) if k.startswith("mat") else (64,), k.split(":")[1]) for k in kinds]
        keep = trace(d.ctx, ins, 64)
        out.append((name, d.keys()))
    # reductions of a computed value: the program whose kernel reduces instead of storing (planned as such only when a
    # kernel for it exists: here the run-time specialiser builds one while planning; shapes large enough for two stages)
    for name, kinds, trace in idioms.REDUCED:
        d = Dry(specialise=1)
        ins = [d.leaf((4096, 64), k.split(":")[1]) for k in kinds]
        keep = trace(d.ctx, ins, 64)
        keys = [k for k in d.keys() if any(int(c) >= 8 for c in k.split("|")[2].split())]
        assert len(keys) == 1, (name, keys)
        out.append((name, keys))
    d = Dry()
    shapes = [(64,), (128,)]
    P, G, Bf = ([d.leaf(s, "f32") for s in shapes] for _ in range(3))
    idioms.sgd_momentum(d.ctx, P, G, Bf)
    out.append(("sgd_momentum", d.keys()))
    # every single-op program of the five configurations traced with fusion off: the unfused baseline
    # ("one kernel per traced op") then runs compiled kernels too, not the interpreter
    for name, record in unfused_traces():
        d = Dry(fusion=0)
        keep = record(d)
        out.append((name, d.keys()))
    del keep
    return out


def unfused_traces():
    def c1(d):
        return traces.elementwise_chain(d.ctx, *(d.leaf((64, 64), "f32") for _ in range(4)))

    def c2(d, prim):
        x, h = (d.leaf((16, 64), "bf16") for _ in range(2))
        return traces.mlp_epilogue(d.ctx, x, h, d.leaf((64,), "bf16"), primitive_gelu=prim)

    def c3(d):
        x, h = (d.leaf((16, 64), "bf16") for _ in range(2))
        g, be = (d.leaf((64,), "f32") for _ in range(2))
        return traces.residual_dropout_layernorm(d.ctx, x, h, g, be, shape=(16, 64), p=0.1, eps=1e-5, seed=1, offset=0)

    def c4(d):
        return traces.causal_softmax(d.ctx, d.leaf((2, 64, 64), "bf16"), shape=(2, 64, 64), scale=0.1)

    def c5(d):
        shapes = [(64,), (128,)]
        P, G, M, V = ([d.leaf(s, "f32") for s in shapes] for _ in range(4))
        traces.adam_step(d.ctx, P, G, M, V, step=1)
        return P

    return [("op_c1", c1), ("op_c2", lambda d: c2(d, False)), ("op_c2p", lambda d: c2(d, True)), ("op_c3", c3),
            ("op_c4", c4), ("op_c5", c5)]


def parse(key: str):
    head, dts, cls, ins = (part.split() for part in key.split("|"))
    kind, flavour, n_pro = (int(v) for v in head)
    return kind, flavour, n_pro, [int(v) for v in dts], [int(v) for v in cls], [tuple(int(x) for x in i.split(":")) for i in ins]


def check(name, kind, n_pro, cls, ins):
    """What the compiled shells assume about a program (anything else stays on the interpreter)."""
    reserved = set()
    for op, slot in ins[:n_pro]:
        d = op - OP_LD
        assert 0 <= d < NT and cls[slot] != 0, f"{name}: prologue must load broadcast operands into temporaries"
        reserved.add(d)
    for op, imm in ins[n_pro:]:
        assert not (OP_MOV_T_ACC <= op < OP_MOV_T_ACC + NT and op - OP_MOV_T_ACC in reserved), f"{name}: reserved temporary overwritten"
        assert not (OP_LD <= op < OP_LD + NT and op - OP_LD in reserved), f"{name}: reserved temporary overwritten"
        if op == OP_ST:
            assert cls[imm] in (0, 2) or (kind == 0 and cls[imm] >= 8), f"{name}: compiled kernels store full-class results, one value per row, or reduce"


def render() -> tuple[str, list[str]]:
    """Text of compiled_programs.inc for the programs the planner emits today, and the entry names."""
    seen = {}
    for name, keys in programs():
        for i, key in enumerate(keys):
            if key not in seen:
                seen[key] = name if len(keys) == 1 else f"{name}_{i}"
    lines = ["// Generated by gen_compiled.py -- do not edit.  One struct per program with an ahead-of-time compiled kernel.", ""]
    names = []
    for n, (key, name) in enumerate(seen.items()):
        kind, flavour, n_pro, dts, cls, ins = parse(key)
        check(name, kind, n_pro, cls, ins)
        cname = f"CP{n}_{name}"
        names.append(cname)
        lines += [
            f"struct {cname} {{",
            f'    static constexpr const char *name = "{name}";',
            f"    static constexpr int kind = {kind}, flavour = {flavour}, n_pro = {n_pro}, n_ins = {len(ins)}, n_slots = {len(dts)};",
            f"    static constexpr LtIns ins[{len(ins)}] = {{" + ", ".join(f"{{{o}, {i}}}" for o, i in ins) + "};",
            f"    static constexpr uint8_t dtype[{len(dts)}] = {{" + ", ".join(map(str, dts)) + "};",
            f"    static constexpr uint8_t cls[{len(cls)}] = {{" + ", ".join(map(str, cls)) + "};",
            "};",
            "",
        ]
    lines.append("#define LT_COMPILED_LIST(X) " + " ".join(f"X({c})" for c in names))
    return "\n".join(lines) + "\n", names


def main() -> None:
    text, names = render()
    (HERE / "compiled_programs.inc").write_text(text)
    print(f"{len(names)} programs:", ", ".join(names))


if __name__ == "__main__":
    main()
