#!/usr/bin/env python
"""Generates vm_core.inc: the interpreter core of the fused-group kernels, as inline PTX.

nvcc lowers a C++ `switch` over the opcode space to a tree of compares and branches (a dozen
branches per interpreted instruction).  Written in PTX instead, the dispatch is one indexed
branch (`brx.idx`) through a table with one entry per opcode, and the twenty 64-bit operands of
the asm statement are the machine state: ACC and T0..T3, eight f32 lanes each, held as four
register pairs so that add/sub/mul/fma run as packed `.f32x2` instructions.

The core executes register-to-register opcodes, the aligned full-chunk loads and stores (from
global memory or from the thread's staging buffer) and, for the elementwise kernel, the loop over
the thread's chunks with its asynchronous staging copies.  Everything else (ragged or unaligned
chunks, broadcast loads, reductions, random bits, correctly rounded transcendentals) leaves the
asm statement with the opcode in an output operand ("escape") and is handled by the surrounding
C++.

Run `python gen_vm_core.py` after changing vm.h's opcode map; the output is committed.
"""
from __future__ import annotations

import re
import struct
from pathlib import Path

HERE = Path(__file__).resolve().parent


def opcodes() -> dict[str, int]:
    """Opcode bases and indices, read from vm.h so the two cannot drift apart."""
    text = (HERE / "vm.h").read_text()
    vals: dict[str, int] = {}
    for m in re.finditer(r"#define\s+(LT_VM_\w+)\s+(\d+)", text):
        vals[m.group(1)] = int(m.group(2))
    for block in re.findall(r"enum\s*\{(.*?)\};", text, flags=re.S):
        block = re.sub(r"/\*.*?\*/", "", block, flags=re.S)
        block = re.sub(r"//[^\n]*", "", block)
        nxt = 0
        for item in block.split(","):
            item = item.strip()
            if not item:
                continue
            if "=" in item:
                name, expr = (s.strip() for s in item.split("=", 1))
                nxt = int(eval(expr, {}, vals))
            else:
                name = item
            vals[name] = nxt
            nxt += 1
    for m in re.finditer(r"#define\s+(LT_VM_\w+)\s+(\d+)", text):
        vals[m.group(1)] = int(m.group(2))
    return vals


OPS = opcodes()
NSRC, NT, ND = OPS["LT_VM_NSRC"], OPS["LT_VM_NT"], OPS["LT_VM_ND"]

A = [f"%{i}" for i in range(4)]
T = [[f"%{4 + 4 * k + j}" for j in range(4)] for k in range(NT)]
REG = T + [A]  # destination index < NT = temporaries, NT = ACC
_o = 4 + 4 * NT
PC, EOP, EIMM, CHUNK, OFF4, COFF4, TAIL, STG, SMB = (f"%{_o + i}" for i in range(9))
PF4 = "pf4"
SM_SCAL, SM_PTR, SM_SOFF, STAGE_PIECE, SM_LOOP, SM_STG = (OPS[k] for k in ("LT_VM_SM_SCAL", "LT_VM_SM_PTR", "LT_VM_SM_SOFF", "LT_VM_STAGE_PIECE", "LT_VM_SM_LOOP", "LT_VM_SM_STG"))
SM_PF = SM_STG + 16 * OPS["LT_VM_MAX_PTR"]


def f32_hex(x: float) -> int:
    return struct.unpack("<I", struct.pack("<f", x))[0]


def pair_imm(x: float) -> str:
    h = f32_hex(x)
    return f"0x{h:08X}{h:08X}"


def const_pair(reg: str, x: float) -> str:
    return f"mov.b64 {reg}, {pair_imm(x)};"


def unpack(pairs, names):
    return [f"mov.b64 {{{names[2 * j]}, {names[2 * j + 1]}}}, {pairs[j]};" for j in range(4)]


def pack(pairs, names):
    return [f"mov.b64 {pairs[j]}, {{{names[2 * j]}, {names[2 * j + 1]}}};" for j in range(4)]


X = [f"x{i}" for i in range(8)]
Y = [f"y{i}" for i in range(8)]
M = [f"m{i}" for i in range(8)]


class Src:
    """Second operand of a two-operand opcode: a temporary or a broadcast immediate."""

    def __init__(self, kind: int):
        self.kind = kind
        if kind < NT:
            self.pre = []
            self.pairs = T[kind]
        else:
            self.pre = ["shl.b32 sa, imm, 2;", f"add.u32 sa, sa, {SMB};", f"ld.shared.b32 sv, [sa+{SM_SCAL}];", "mov.b64 ss, {sv, sv};"]
            self.pairs = ["ss"] * 4


def div_ins(flavour: str) -> str:
    # fast: rcp-and-multiply; precise: full-range division within 2 ulp; ieee: correctly rounded
    return {"fast": "div.approx.f32", "precise": "div.full.f32", "ieee": "div.rn.f32"}[flavour]


def pairwise(a_pairs, src, fmt_lines):
    """Lane-by-lane op on ACC done one register pair at a time (keeps few registers live).
    fmt_lines(x, y) -> PTX lines computing x = op(x, y) for one lane."""
    lines = []
    for j in range(4):
        lines.append(f"mov.b64 {{x0, x1}}, {a_pairs[j]};")
        if src is None:
            ys = (None, None)
        elif src.kind < NT:
            lines.append(f"mov.b64 {{y0, y1}}, {src.pairs[j]};")
            ys = ("y0", "y1")
        else:
            ys = ("sv", "sv")
        lines += fmt_lines("x0", ys[0]) + fmt_lines("x1", ys[1])
        lines.append(f"mov.b64 {a_pairs[j]}, {{x0, x1}};")
    return lines


def f2_body(idx: int, src: Src, flavour: str):
    names = ["add", "sub", "rsub", "mul", "div", "rdiv", "max", "min"]
    op = names[idx]
    lines = list(src.pre)
    if op in ("add", "sub", "mul"):
        lines += [f"{op}.rn.f32x2 {A[j]}, {A[j]}, {src.pairs[j]};" for j in range(4)]
    elif op == "rsub":
        lines += [f"sub.rn.f32x2 {A[j]}, {src.pairs[j]}, {A[j]};" for j in range(4)]
    elif op == "div":
        lines += pairwise(A, src, lambda x, y: [f"{div_ins(flavour)} {x}, {x}, {y};"])
    elif op == "rdiv":
        lines += pairwise(A, src, lambda x, y: [f"{div_ins(flavour)} {x}, {y}, {x};"])
    else:
        lines += pairwise(A, src, lambda x, y: [f"{op}.NaN.f32 {x}, {x}, {y};"])
    return lines


def i2_body(idx: int, src: Src):
    ops = ["add.s32", "sub.s32", "rsub", "mul.lo.s32", "and.b32", "or.b32", "xor.b32", "max.s32", "min.s32", "max.u32", "min.u32"]
    op = ops[idx]
    if op == "rsub":
        return list(src.pre) + pairwise(A, src, lambda x, y: [f"sub.s32 {x}, {y}, {x};"])
    return list(src.pre) + pairwise(A, src, lambda x, y: [f"{op} {x}, {x}, {y};"])


def cmp_body(idx: int, src: Src):
    ty, cc = divmod(idx, 6)
    ccn = ["gt", "ge", "lt", "le", "eq", "ne"][cc]
    if ty == 0:
        ins = f"setp.{'neu' if ccn == 'ne' else ccn}.f32"
    elif ty == 1:
        ins = f"setp.{ccn}.s32"
    else:
        ins = f"setp.{ {'gt': 'hi', 'ge': 'hs', 'lt': 'lo', 'le': 'ls', 'eq': 'eq', 'ne': 'ne'}[ccn] }.u32"
    return list(src.pre) + pairwise(A, src, lambda x, y: [f"{ins} p, {x}, {y};", f"selp.b32 {x}, 1, 0, p;"])


def where_body(m: int, src: Src, variant_b: bool):
    lines = list(src.pre)
    for j in range(4):
        lines += [f"mov.b64 {{x0, x1}}, {A[j]};", f"mov.b64 {{m0, m1}}, {T[m][j]};"]
        if src.kind < NT:
            lines.append(f"mov.b64 {{y0, y1}}, {src.pairs[j]};")
            ys = ("y0", "y1")
        else:
            ys = ("sv", "sv")
        for x, mm, y in (("x0", "m0", ys[0]), ("x1", "m1", ys[1])):
            lines.append(f"setp.ne.u32 p, {mm}, 0;")
            lines.append(f"selp.b32 {x}, {y}, {x}, p;" if variant_b else f"selp.b32 {x}, {x}, {y}, p;")
        lines.append(f"mov.b64 {A[j]}, {{x0, x1}};")
    return lines


LOG2E, LN2 = 1.4426950408889634, 0.6931471805599453
GELU_K = 0.7978845608028654
GELU_KC = GELU_K * 0.044715


def lanes_op(fmt: str):
    return pairwise(A, None, lambda x, y: [fmt.format(x=x)])


def unary_body(name: str, flavour: str):
    fast = flavour == "fast"
    ieee = flavour == "ieee"
    """Returns PTX lines, or None when the opcode escapes to C++ in this flavour."""
    if name == "OP_U_NEG":
        return [f"xor.b64 {a}, {a}, 0x8000000080000000;" for a in A]
    if name == "OP_U_ABS":
        return [f"and.b64 {a}, {a}, 0x7FFFFFFF7FFFFFFF;" for a in A]
    if name == "OP_U_RELU":
        return lanes_op("max.NaN.f32 {x}, {x}, 0f00000000;")
    if name == "OP_U_SQUARE":
        return [f"mul.rn.f32x2 {a}, {a}, {a};" for a in A]
    if name == "OP_U_SQRT":
        return lanes_op("sqrt.rn.f32 {x}, {x};" if ieee else "sqrt.approx.f32 {x}, {x};")
    if name == "OP_U_RSQRT":
        return lanes_op("rsqrt.approx.f32 {x}, {x};")
    if name == "OP_U_RECIP":
        return lanes_op("rcp.rn.f32 {x}, {x};" if ieee else ("rcp.approx.ftz.f32 {x}, {x};" if fast else "rcp.approx.f32 {x}, {x};"))
    if name == "OP_U_RBF16":
        lines = []
        for j in range(4):
            lines += [f"mov.b64 {{x0, x1}}, {A[j]};", "cvt.rn.bf16x2.f32 w0, x1, x0;", "shl.b32 x0, w0, 16;",
                      "and.b32 x1, w0, 0xFFFF0000;", f"mov.b64 {A[j]}, {{x0, x1}};"]
        return lines
    if name == "OP_U_INEG":
        return lanes_op("neg.s32 {x}, {x};")
    if name == "OP_U_IABS":
        return lanes_op("abs.s32 {x}, {x};")
    if name == "OP_U_NOT":
        return pairwise(A, None, lambda x, y: [f"setp.eq.u32 p, {x}, 0;", f"selp.b32 {x}, 1, 0, p;"])
    if name == "OP_C_I2F":
        return lanes_op("cvt.rn.f32.s32 {x}, {x};")
    if name == "OP_C_U2F":
        return lanes_op("cvt.rn.f32.u32 {x}, {x};")
    if name == "OP_C_F2I":
        return lanes_op("cvt.rzi.s32.f32 {x}, {x};")
    if name == "OP_C_NZF":
        return pairwise(A, None, lambda x, y: [f"setp.neu.f32 p, {x}, 0f00000000;", f"selp.b32 {x}, 1, 0, p;"])
    if name == "OP_C_NZI":
        return pairwise(A, None, lambda x, y: [f"setp.ne.u32 p, {x}, 0;", f"selp.b32 {x}, 1, 0, p;"])
    if not fast:
        return None  # exp, log, tanh, sigmoid, gelu: correctly rounded versions live in C++
    if name == "OP_U_EXP":
        return ([const_pair("c0", LOG2E)] + [f"mul.rn.f32x2 {a}, {a}, c0;" for a in A] + lanes_op("ex2.approx.ftz.f32 {x}, {x};"))
    if name == "OP_U_LOG":
        return lanes_op("lg2.approx.f32 {x}, {x};") + [const_pair("c0", LN2)] + [f"mul.rn.f32x2 {a}, {a}, c0;" for a in A]
    if name == "OP_U_TANH":
        return lanes_op("tanh.approx.f32 {x}, {x};")
    if name == "OP_U_SIGMOID":
        lines = [const_pair("c0", -LOG2E), const_pair("c1", 1.0)] + [f"mul.rn.f32x2 {a}, {a}, c0;" for a in A]
        lines += lanes_op("ex2.approx.ftz.f32 {x}, {x};")
        lines += [f"add.rn.f32x2 {a}, {a}, c1;" for a in A]
        return lines + lanes_op("rcp.approx.ftz.f32 {x}, {x};")
    if name == "OP_U_GELU":
        lines = [const_pair("c0", GELU_KC), const_pair("c1", GELU_K), const_pair("c2", 0.5)]
        for j, a in enumerate(A):
            g = "g0"
            lines += [f"mul.rn.f32x2 {g}, {a}, {a};",
                      f"fma.rn.f32x2 {g}, {g}, c0, c1;",
                      f"mul.rn.f32x2 {g}, {g}, {a};",
                      f"mov.b64 {{x0, x1}}, {g};", "tanh.approx.f32 x0, x0;", "tanh.approx.f32 x1, x1;",
                      f"mov.b64 {g}, {{x0, x1}};",
                      f"mul.rn.f32x2 {a}, {a}, c2;",
                      f"fma.rn.f32x2 {a}, {a}, {g}, {a};"]
        return lines
    raise KeyError(name)


def slot_address(cls: int, sz: int, prefetch: bool):
    """ptr = address of this thread's chunk in pointer slot `imm` (the slot was linked as vector-capable)."""
    lines = ["@ptail bra L_ESC;", "shl.b32 sa, imm, 3;", f"add.u32 sa, sa, {SMB};", f"ld.shared.b64 ptr, [sa+{SM_PTR}];",
             "setp.lt.s64 p, ptr, 0;", "@p bra L_ESC;"]  # bit 63: this pointer cannot take vector accesses after all
    if cls == 0:
        lines.append(f"shr.u64 offs, {OFF4}, {sz};" if sz else f"mov.b64 offs, {OFF4};")
    else:
        lines += [f"cvt.u64.u32 offs, {COFF4};"] + ([f"shr.u64 offs, offs, {sz};"] if sz else [])
    lines.append("add.u64 ptr, ptr, offs;")
    if prefetch and cls == 0:
        # pull this thread's next chunk of the same input into L2 while the current one is processed
        lines += [f"@pnext ld.shared.b64 offs, [{SMB}+{SM_PF}];"] + ([f"@pnext shr.u64 offs, offs, {sz};"] if sz else []) + [
                  "@pnext add.u64 offs, ptr, offs;", "@pnext prefetch.global.L2 [offs];"]
    return lines


def raw_load(sz: int, space: str, addr: str):
    """Raw chunk into x0.. : 8 words (4-byte elements), 4 words (2-byte) or 2 words (1-byte)."""
    if sz == 0:
        return [f"{space}.v4.b32 {{x0, x1, x2, x3}}, [{addr}];", f"{space}.v4.b32 {{x4, x5, x6, x7}}, [{addr}+{16 if 'global' in space else STAGE_PIECE}];"]
    if sz == 1:
        return [f"{space}.v4.b32 {{x0, x1, x2, x3}}, [{addr}];"]
    return [f"{space}.v2.b32 {{x0, x1}}, [{addr}];"]


def widened_pair(sz: int, j: int, dst: str):
    """PTX putting lanes 2j, 2j+1 of the raw chunk in x0.. into the 64-bit register `dst` as 32-bit lanes."""
    if sz == 0:
        return [f"mov.b64 {dst}, {{x{2 * j}, x{2 * j + 1}}};"]
    if sz == 1:
        return [f"shl.b32 y0, x{j}, 16;", f"and.b32 y1, x{j}, 0xFFFF0000;", f"mov.b64 {dst}, {{y0, y1}};"]
    w, k = divmod(2 * j, 4)
    return [f"bfe.u32 y0, x{w}, {8 * k}, 8;", f"bfe.u32 y1, x{w}, {8 * k + 8}, 8;", f"mov.b64 {dst}, {{y0, y1}};"]


def ldg_body(sz: int, cls: int, d: int):
    space = "ld.global.cs" if cls == 0 else "ld.global.nc"
    lines = slot_address(cls, sz, True) + raw_load(sz, space, "ptr")
    for j in (3, 2, 1, 0):
        lines += widened_pair(sz, j, REG[d][j])
    return lines


def lds_body(sz: int, d: int):
    lines = ["@ptail bra L_ESC;", f"add.u32 w0, imm, {STG};"] + raw_load(sz, "ld.shared", "w0")
    for j in (3, 2, 1, 0):
        lines += widened_pair(sz, j, REG[d][j])
    return lines


def f2m_tail(k: int, sz: int):
    op = ["add", "sub", "rsub", "mul"][k]
    lines = []
    for j in range(4):
        lines += widened_pair(sz, j, "g0")
        lines.append(f"sub.rn.f32x2 {A[j]}, g0, {A[j]};" if op == "rsub" else f"{op}.rn.f32x2 {A[j]}, {A[j]}, g0;")
    return lines


def f2mg_body(k: int, sz: int, cls: int):
    space = "ld.global.cs" if cls == 0 else "ld.global.nc"
    return slot_address(cls, sz, True) + raw_load(sz, space, "ptr") + f2m_tail(k, sz)


def f2ms_body(k: int, sz: int):
    return ["@ptail bra L_ESC;", f"add.u32 w0, imm, {STG};"] + raw_load(sz, "ld.shared", "w0") + f2m_tail(k, sz)


def stg_body(sz: int):
    lines = slot_address(0, sz, False) + unpack(A, X)
    if sz == 0:
        lines += ["st.global.cs.v4.b32 [ptr], {x0, x1, x2, x3};", "st.global.cs.v4.b32 [ptr+16], {x4, x5, x6, x7};"]
    elif sz == 1:
        for j in range(4):
            lines.append(f"cvt.rn.bf16x2.f32 w{j}, {X[2 * j + 1]}, {X[2 * j]};")
        lines.append("st.global.cs.v4.b32 [ptr], {w0, w1, w2, w3};")
    else:
        for h in range(2):
            b = 4 * h
            lines += [f"prmt.b32 y0, {X[b]}, {X[b + 1]}, 0x0040;", f"prmt.b32 y1, {X[b + 2]}, {X[b + 3]}, 0x0040;",
                      f"prmt.b32 w{h}, y0, y1, 0x5410;"]
        lines.append("st.global.cs.v2.b32 [ptr], {w0, w1};")
    return lines


SM_N4 = SM_PF + 8
SM_GROUP = SM_PF + 16
SM_RED = OPS["LT_VM_SM_RED"]
SM_DPF = SM_PF + 24


def entry_code():
    """Registers that depend on the current chunk or thread; recomputed whenever the asm statement is
    (re-)entered.  TAIL bits: 1 = this chunk is ragged or absent, 2 = the thread's column range is never a
    full chunk (row kernel), 4 = which half of the reduction exchange buffer is next."""
    L = SM_LOOP
    return [f"and.b32 r0, {TAIL}, 1;", "setp.ne.u32 ptail, r0, 0;",
            f"ld.shared.b32 r3, [{SMB}+{L + 12}];",                   # staging depth: which wait_group the loop uses
            "setp.eq.u32 pd1, r3, 1;", "setp.eq.u32 pd2, r3, 2;", "setp.eq.u32 pd3, r3, 3;", "setp.eq.u32 pd4, r3, 4;",
            ] + next_chunk_predicate()


def next_chunk_predicate():
    """pnext: the thread has a further chunk and L2 prefetch is on (full-class vector loads then prefetch it)."""
    L = SM_LOOP
    return [f"ld.shared.v2.b32 {{r0, r1}}, [{SMB}+{L}];",            # stride, n_chunks
            f"ld.shared.b32 r2, [{SMB}+{L + 56}];",                   # prefetch enabled
            f"sub.u32 r1, r1, {CHUNK};", "setp.gt.u32 pnext, r1, r0;", "setp.ne.u32 p, r2, 0;",
            "and.pred pnext, pnext, p;", "not.pred p, ptail;", "and.pred pnext, pnext, p;"]


def stage_loop(label: str, count_shift: int, shift: int):
    """Copies of the staged inputs of one element size (list entries: pointer lo, hi, offset in the buffer).
    With few staging buffers the chunk after the staged one is also pulled into L2 (ppf)."""
    lines = [f"bfe.u32 r8, r9, {count_shift}, 8;", "setp.eq.u32 p, r8, 0;", f"@p bra L_STG_END{label};"]
    if shift == 2:
        lines += ["mov.b64 d1, d0;", "mov.b64 d3, pf4;"]
    else:
        lines += [f"shr.u64 d1, d0, {2 - shift};", f"shr.u64 d3, pf4, {2 - shift};"]   # byte offsets for this element size
    lines += [f"L_STG_LOOP{label}:", "ld.shared.v4.b32 {x0, x1, x2, x3}, [sa];", "mov.b64 ptr, {x0, x1};",
              "add.u64 ptr, ptr, d1;", f"add.u32 x2, x2, {STG};"]
    if shift == 0:
        lines.append("cp.async.ca.shared.global [x2], [ptr], 8;")
    else:
        lines.append("cp.async.cg.shared.global [x2], [ptr], 16;")
        if shift == 2:
            lines.append(f"cp.async.cg.shared.global [x2+{STAGE_PIECE}], [ptr+16], 16;")
    lines += ["@ppf add.u64 ptr, ptr, d3;", "@ppf prefetch.global.L2 [ptr];"]
    lines += ["add.u32 sa, sa, 16;", "sub.u32 r8, r8, 1;", "setp.ne.u32 p, r8, 0;", f"@p bra L_STG_LOOP{label};",
              f"L_STG_END{label}:"]
    return lines


def end_body():
    """OP_END.  When the core runs the loop itself: refill the staging buffer just consumed, move to the
    thread's next chunk (or block of rows), wait for its staged inputs and restart the program."""
    L = SM_LOOP
    lines = [
        f"ld.shared.v4.b32 {{r4, r5, r6, r7}}, [{SMB}+{L + 16}];",     # buf_bytes, buf_total, stage_base, inloop | flags
        "and.b32 x0, r7, 3;", "setp.eq.u32 p, x0, 0;", "@p bra L_ESC;",
        f"ld.shared.v4.b32 {{r0, r1, r2, r3}}, [{SMB}+{L}];",          # stride, n_chunks, body offset, depth
        f"ld.shared.b64 d2, [{SMB}+{SM_N4}];",                          # 4 * elements
        f"ld.shared.b64 pf4, [{SMB}+{SM_PF}];",                         # bytes (4-byte view) between a thread's iterations
        "setp.eq.u32 pq, r3, 0;", "@pq bra L_ADV;",
        # the chunk `depth` iterations ahead, as a byte offset in the 4-byte view; staged if complete
        f"ld.shared.b64 d1, [{SMB}+{SM_DPF}];", f"add.u64 d0, {OFF4}, d1;", "add.u64 d1, d0, 32;",
        "setp.gt.u64 p, d1, d2;", f"and.b32 x0, {TAIL}, 2;", "setp.ne.u32 pq, x0, 0;", "or.pred p, p, pq;",
        "@p bra L_COMMIT;",
        # inloop bit 9: few staging buffers, so the chunk one iteration further is prefetched into L2 (if complete)
        "add.u64 d1, d1, pf4;", "setp.le.u64 ppf, d1, d2;", "and.b32 x0, r7, 512;", "setp.ne.u32 p, x0, 0;",
        "and.pred ppf, ppf, p;",
        f"ld.shared.b32 r9, [{SMB}+{L + 60}];",                         # staged inputs per element size
        f"add.u32 sa, {SMB}, {SM_STG};",
    ]
    lines += stage_loop("4", 0, 2) + stage_loop("2", 8, 1) + stage_loop("1", 16, 0)
    lines += [
        "L_COMMIT:",
        "cp.async.commit_group;",
        # next staging buffer of this thread (a ring of `depth` buffers)
        f"add.u32 {STG}, {STG}, r4;", "mov.u32 x0, %tid.x;", "shl.b32 x0, x0, 4;", "add.u32 x0, x0, r6;",
        "add.u32 x0, x0, r5;", f"setp.ge.u32 p, {STG}, x0;", f"@p sub.u32 {STG}, {STG}, r5;",
        # the copies of the next chunk are the oldest group still in flight
        "@pd3 cp.async.wait_group 2;", "@pd4 cp.async.wait_group 3;", "@pd2 cp.async.wait_group 1;",
        "@pd1 cp.async.wait_group 0;",
        "L_ADV:",
        f"add.u32 {CHUNK}, {CHUNK}, r0;", f"setp.ge.u32 p, {CHUNK}, r1;", "@p bra L_ESC;",
        "and.b32 x0, r7, 3;", "setp.eq.u32 p, x0, 2;", "@p bra L_FIXED;",
        f"ld.shared.v4.b32 {{r4, r5, r6, r9}}, [{SMB}+{L + 32}];",      # rowcol, cpr, div_mul, div_sh1
        "setp.ne.u32 p, r4, 0;", "@p bra L_ROWCOL;",
        # flat chunks: the next chunk of this thread is pf4 bytes further
        f"add.u64 {OFF4}, {OFF4}, pf4;", f"cvt.u32.u64 {COFF4}, {OFF4};", f"add.u64 d1, {OFF4}, 32;",
        "setp.gt.u64 ptail, d1, d2;", "bra L_COORD_DONE;",
        "L_FIXED:",
        # same columns, a fixed distance further (blocks of rows; elementwise rows when the chunk stride is a
        # multiple of the chunks per row); absent once past the last element
        f"add.u64 {OFF4}, {OFF4}, pf4;", f"setp.ge.u64 ptail, {OFF4}, d2;", f"and.b32 x0, {TAIL}, 2;",
        "setp.ne.u32 pq, x0, 0;", "or.pred ptail, ptail, pq;", "bra L_COORD_DONE;",
        "L_ROWCOL:",
        f"ld.shared.v2.b32 {{x2, x3}}, [{SMB}+{L + 48}];",               # div_sh2, cols
        f"mul.hi.u32 x0, r6, {CHUNK};", f"sub.u32 x1, {CHUNK}, x0;", "shr.u32 x1, x1, r9;", "add.u32 x0, x0, x1;",
        "shr.u32 x0, x0, x2;",                                           # row
        f"mul.lo.u32 x1, x0, r5;", f"sub.u32 x1, {CHUNK}, x1;", "shl.b32 x1, x1, 3;",   # col0
        "mul.wide.u32 d0, x0, x3;", "cvt.u64.u32 d1, x1;", "add.u64 d0, d0, d1;", f"shl.b64 {OFF4}, d0, 2;",
        f"shl.b32 {COFF4}, x1, 2;", "sub.u32 x1, x3, x1;", "setp.lt.u32 ptail, x1, 8;",
        "L_COORD_DONE:",
        f"and.b32 {TAIL}, {TAIL}, 0xFFFFFFFE;", "selp.b32 x0, 1, 0, ptail;", f"or.b32 {TAIL}, {TAIL}, x0;",
        f"add.u32 {PC}, {SMB}, r2;",                                    # restart after the once-per-thread part
        # L2 prefetch is off whenever inputs are staged: only then is pnext worth recomputing
        "and.b32 x0, r7, 256;", "setp.eq.u32 pnext, x0, 0;", "@pnext bra L_NO_PF;",
    ] + next_chunk_predicate() + ["bra L_RESTART;", "L_NO_PF:", "setp.ne.u32 pnext, x0, 0;", "L_RESTART:",
                                  f"ld.shared.v2.b32 {{nop, nimm}}, [{PC}];"]
    return lines


def inline_rows_guard():
    """Row-wise opcodes run in the core only when rows are regular (see LtLoop::inline_rows) and the chunk
    is complete where that matters."""
    return [f"ld.shared.v2.b32 {{r0, r1}}, [{SMB}+{SM_GROUP}];", "setp.eq.u32 p, r1, 0;", "@p bra L_ESC;"]


def red_body(kind: int):
    """ACC = reduction of the row, broadcast: lanes of the thread, then shuffles within the warp, then (rows
    wider than a warp's 256 elements) one exchange through shared memory."""
    op = ["add.rn.f32", "max.NaN.f32", "min.NaN.f32"][kind]
    ident = ["0f00000000", "0fFF800000", "0f7F800000"][kind]   # 0, -inf, +inf
    lines = inline_rows_guard()          # r0 = threads per row
    lines += unpack(A, X)
    lines += [f"{op} x0, x0, x1;", f"{op} x2, x2, x3;", f"{op} x4, x4, x5;", f"{op} x6, x6, x7;",
              f"{op} x0, x0, x2;", f"{op} x4, x4, x6;", f"{op} x0, x0, x4;"]
    for off in (16, 8, 4, 2, 1):
        lines += [f"setp.gt.u32 p, r0, {off};", f"@p shfl.sync.bfly.b32 y0, x0, {off}, 0x1f, 0xffffffff;",
                  f"@p {op} x0, x0, y0;"]
    lines += [
        "setp.le.u32 p, r0, 32;", f"@p bra L_RED_DONE{kind};",
        "mov.u32 r2, %tid.x;", "shr.u32 r3, r2, 5;", "and.b32 r2, r2, 31;",          # r3 warp, r2 lane
        f"and.b32 r4, {TAIL}, 4;", "shl.b32 r4, r4, 5;", f"add.u32 r4, r4, {SMB};",   # half of the exchange buffer
        "shl.b32 r5, r3, 2;", "add.u32 r5, r5, r4;", "setp.eq.u32 p, r2, 0;", f"@p st.shared.b32 [r5+{SM_RED}], x0;",
        "bar.sync 0;",
        # r6 = warps per row (a power of two <= 32), r7 = first warp of this row: lane l < r6 takes that
        # warp's partial, the others the identity, and a shuffle tree combines them
        "shr.u32 r6, r0, 5;", "sub.u32 r7, r6, 1;", "not.b32 r7, r7;", "and.b32 r7, r3, r7;",
        "add.u32 r7, r7, r2;", "shl.b32 r7, r7, 2;", "add.u32 r7, r7, r4;",
        f"mov.b32 x0, {ident};", "setp.lt.u32 p, r2, r6;", f"@p ld.shared.b32 x0, [r7+{SM_RED}];",
        "setp.gt.u32 p, r6, 16;", "@p shfl.sync.bfly.b32 y0, x0, 16, 0x1f, 0xffffffff;", f"@p {op} x0, x0, y0;",
        "setp.gt.u32 p, r6, 8;", "@p shfl.sync.bfly.b32 y0, x0, 8, 0x1f, 0xffffffff;", f"@p {op} x0, x0, y0;",
        "setp.gt.u32 p, r6, 4;", "@p shfl.sync.bfly.b32 y0, x0, 4, 0x1f, 0xffffffff;", f"@p {op} x0, x0, y0;",
        "setp.gt.u32 p, r6, 2;", "@p shfl.sync.bfly.b32 y0, x0, 2, 0x1f, 0xffffffff;", f"@p {op} x0, x0, y0;",
        "setp.gt.u32 p, r6, 1;", "@p shfl.sync.bfly.b32 y0, x0, 1, 0x1f, 0xffffffff;", f"@p {op} x0, x0, y0;",
        "shfl.sync.idx.b32 x0, x0, 0, 0x1f, 0xffffffff;",   # lanes past the row's warp count hold the identity only
        f"xor.b32 {TAIL}, {TAIL}, 4;",
        f"L_RED_DONE{kind}:",
    ]
    lines += [f"mov.b64 {a}, {{x0, x0}};" for a in A]
    return lines


def iota_row_body():
    """ACC = (row / scal[imm]) % scal[imm+1]; the row is recovered from the chunk's byte offsets: rows are a
    multiple of the chunk here, so row = (chunks before this row's start) / (chunks per row), by multiply-shift."""
    L = SM_LOOP
    return inline_rows_guard() + [
        f"cvt.u64.u32 d0, {COFF4};", f"sub.u64 d0, {OFF4}, d0;", "shr.u64 d0, d0, 5;", "cvt.u32.u64 x0, d0;",   # row * chunks per row
        f"ld.shared.v2.b32 {{x1, x2}}, [{SMB}+{L + 40}];", f"ld.shared.b32 x3, [{SMB}+{L + 48}];",              # div_mul, div_sh1, div_sh2
        "mul.hi.u32 x4, x1, x0;", "sub.u32 x5, x0, x4;", "shr.u32 x5, x5, x2;", "add.u32 x4, x4, x5;", "shr.u32 x0, x4, x3;",  # row
        "shl.b32 sa, imm, 2;", f"add.u32 sa, sa, {SMB};", f"ld.shared.b32 x1, [sa+{SM_SCAL}];",
        f"ld.shared.b32 x2, [sa+{SM_SCAL + 4}];",   # two loads: the slot pair need not be 8-byte aligned
        "setp.ne.u32 p, x1, 1;", "@p div.u32 x0, x0, x1;",
        "sub.u32 x3, x2, 1;", "and.b32 x4, x3, x2;", "setp.eq.u32 p, x4, 0;",                                   # extent a power of two?
        "@p and.b32 x0, x0, x3;", "@!p rem.u32 x0, x0, x2;",
    ] + [f"mov.b64 {a}, {{x0, x0}};" for a in A]


def philox_body():
    """ACC = Philox4x32-10 bits of the chunk's eight elements (two counter blocks; Salmon et al., SC'11)."""
    lines = inline_rows_guard()[:0] + ["@ptail bra L_ESC;", "shl.b32 sa, imm, 2;", f"add.u32 sa, sa, {SMB};",
             f"ld.shared.v2.b32 {{r0, r1}}, [sa+{SM_SCAL}];", f"ld.shared.v2.b32 {{r2, r3}}, [sa+{SM_SCAL + 8}];",
             f"shr.u64 d0, {OFF4}, 4;"]                                   # block index q = element / 4 (a complete chunk starts a block)
    for blk in range(2):
        lines += ["mov.b64 {x0, x1}, d0;", "mov.b32 x2, r2;", "mov.b32 x3, r3;", "mov.b32 y0, r0;", "mov.b32 y1, r1;"]
        for rnd in range(10):
            lines += ["mul.hi.u32 x4, x0, 0xD2511F53;", "mul.lo.u32 x5, x0, 0xD2511F53;",
                      "mul.hi.u32 x6, x2, 0xCD9E8D57;", "mul.lo.u32 x7, x2, 0xCD9E8D57;",
                      "xor.b32 x0, x6, x1;", "xor.b32 x0, x0, y0;", "mov.b32 x1, x7;",
                      "xor.b32 x2, x4, x3;", "xor.b32 x2, x2, y1;", "mov.b32 x3, x5;"]
            if rnd < 9:
                lines += ["add.u32 y0, y0, 0x9E3779B9;", "add.u32 y1, y1, 0xBB67AE85;"]
        lines += [f"mov.b64 {A[2 * blk]}, {{x0, x1}};", f"mov.b64 {A[2 * blk + 1]}, {{x2, x3}};", "add.u64 d0, d0, 1;"]
    return lines


def build(flavour: str) -> list[str]:
    limit = OPS["OP_LIMIT"]
    bodies: dict[int, list[str]] = {}

    bodies[OPS["OP_END"]] = end_body()
    for kind in range(3):
        bodies[OPS["OP_RED_SUM"] + kind] = red_body(kind)
    bodies[OPS["OP_IOTA_ROW"]] = iota_row_body()
    bodies[OPS["OP_PHILOX"]] = philox_body()
    for k in range(NT):
        bodies[OPS["OP_MOV_T_ACC"] + k] = [f"mov.b64 {T[k][j]}, {A[j]};" for j in range(4)]
        bodies[OPS["OP_MOV_ACC_T"] + k] = [f"mov.b64 {A[j]}, {T[k][j]};" for j in range(4)]
    s = Src(NT)
    bodies[OPS["OP_MOV_ACC_S"]] = s.pre + [f"mov.b64 {a}, ss;" for a in A]
    bodies[OPS["OP_IOTA_COL"]] = ([f"shr.u32 w0, {COFF4}, 2;"] + [f"add.u32 {X[i]}, w0, {i};" for i in range(8)] + pack(A, X))
    for name in ("OP_U_NEG", "OP_U_ABS", "OP_U_RELU", "OP_U_EXP", "OP_U_LOG", "OP_U_TANH", "OP_U_SQRT", "OP_U_RSQRT",
                 "OP_U_RECIP", "OP_U_SQUARE", "OP_U_SIGMOID", "OP_U_GELU", "OP_U_RBF16", "OP_U_INEG", "OP_U_IABS",
                 "OP_U_NOT", "OP_C_I2F", "OP_C_U2F", "OP_C_F2I", "OP_C_NZF", "OP_C_NZI"):
        b = unary_body(name, flavour)
        if b is not None:
            bodies[OPS[name]] = b
    for sz in range(3):
        for d in range(ND):
            for cls in range(2):
                bodies[OPS["OP_LDG"] + (sz * 2 + cls) * ND + d] = ldg_body(sz, cls, d)
            bodies[OPS["OP_LDS"] + sz * ND + d] = lds_body(sz, d)
        bodies[OPS["OP_STG"] + sz] = stg_body(sz)
        for k in range(OPS["F2M_COUNT"]):
            for cls in range(2):
                bodies[OPS["OP_F2MG"] + (k * 3 + sz) * 2 + cls] = f2mg_body(k, sz, cls)
            bodies[OPS["OP_F2MS"] + k * 3 + sz] = f2ms_body(k, sz)
    for idx in range(OPS["F2_COUNT"]):
        for k in range(NSRC):
            bodies[OPS["OP_F2"] + idx * NSRC + k] = f2_body(idx, Src(k), flavour)
    for idx in range(OPS["I2_COUNT"]):
        for k in range(NSRC):
            bodies[OPS["OP_I2"] + idx * NSRC + k] = i2_body(idx, Src(k))
    for idx in range(OPS["CMP_COUNT"]):
        for k in range(NSRC):
            bodies[OPS["OP_CMP"] + idx * NSRC + k] = cmp_body(idx, Src(k))
    for m in range(NT):
        for k in range(NSRC):
            bodies[OPS["OP_WHERE_A"] + m * NSRC + k] = where_body(m, Src(k), False)
            bodies[OPS["OP_WHERE_B"] + m * NSRC + k] = where_body(m, Src(k), True)

    out = ["{"]
    out.append(".reg .b32 op, imm, nop, nimm, sa, sv, w0, w1, w2, w3, r0, r1, r2, r3, r4, r5, r6, r7, r8, r9;")
    out.append(".reg .b32 " + ", ".join(X + ["y0", "y1", "m0", "m1"]) + ";")
    out.append(".reg .b64 ss, ptr, offs, g0, c0, c1, c2, d0, d1, d2, d3, pf4;")
    out.append(".reg .pred p, pq, ptail, pnext, ppf, pd1, pd2, pd3, pd4;")
    table = ", ".join(f"L_{i}" if i in bodies else "L_ESC" for i in range(limit))
    out.append(f"TBL: .branchtargets {table};")
    out += entry_code()
    out.append(f"ld.shared.v2.b32 {{nop, nimm}}, [{PC}];")
    # fetch/decode/jump.  The next instruction word is fetched one step ahead (the slot after the last
    # instruction is padding).
    dispatch = ["mov.b32 op, nop;", "mov.b32 imm, nimm;", f"add.u32 {PC}, {PC}, 8;",
                f"ld.shared.v2.b32 {{nop, nimm}}, [{PC}];", "brx.idx op, TBL;"]
    # One shared copy: replicating the indexed branch after every body saves a jump per instruction but
    # gives ptxas ~300 indirect branches x 328 targets to analyse, and compile time goes from seconds
    # to tens of minutes.
    out.append("L_DISPATCH:")
    out += dispatch
    for code in sorted(bodies):
        out.append(f"L_{code}:")
        for ln in bodies[code]:
            out.append("bra.uni L_DISPATCH;" if ln == "@DISPATCH@" else ln)
        out.append("bra.uni L_DISPATCH;")
    out.append("L_ESC:")
    out.append(f"mov.b32 {EOP}, op;")
    out.append(f"mov.b32 {EIMM}, imm;")
    out.append("}")
    return out


def as_macro(name: str, lines: list[str]) -> str:
    body = " \\\n".join('    "' + ln + '\\n"' for ln in lines)
    return f"#define {name} \\\n{body}\n"


def render() -> str:
    """Text of vm_core.inc for the opcode map vm.h has today."""
    text = ("// Generated by gen_vm_core.py from vm.h -- do not edit.\n"
            f"// Operands: %0-%3 ACC, then the temporaries (f32x2 pairs); {PC} pc (shared address); {EOP} escape opcode;\n"
            f"// {EIMM} escape immediate; {CHUNK} chunk index; {OFF4} chunk byte offset for 4-byte elements; {COFF4} column\n"
            f"// byte offset; {TAIL} chunk flags; {STG} shared address of this thread's current staging buffer;\n"
            f"// {SMB} shared address of the staged block (program, immediates, pointers, loop constants).\n"
            f"// {CHUNK}-{STG} are updated by the core when it moves to the next chunk by itself (OP_END).\n"
            "#pragma once\n\n")
    text += "\n".join(as_macro(f"LT_VM_CORE_{fl.upper()}", build(fl)) for fl in ("fast", "precise", "ieee"))
    return text


def main() -> None:
    text = render()
    (HERE / "vm_core.inc").write_text(text)
    print(f"wrote vm_core.inc ({len(text)} bytes)")


if __name__ == "__main__":
    main()
