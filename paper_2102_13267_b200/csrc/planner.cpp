// Planner: cuts the canonical program into fusion groups, generates each group's register
// program (vm.h), bundles isomorphic independent groups into multi-tensor launches and
// decides which outputs are written into donated input buffers.  This stage takes the
// place of the domain-specific compiler in the paper's pipeline (Section 4); it runs only
// on a compile-cache miss.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <map>

#include "compiled.h"
#include "engine.h"
#include "launch.h"

namespace lt {

namespace {

constexpr int MAX_GROUP_NODES = 64;

struct PNode {
    uint64_t numel = 1, rows = 1, cols = 1;
    int group = -1;      // native group, -1 for leaves and absorbed nodes
    bool leaf = false;   // device data or scalar
    bool absorbed = false;
    bool reduce = false;
    bool in_place_slice = false;  // a narrow of a device-data leaf that its consumers read in place (pitched / offset loads)
    bool foreign = false;  // runs as a kernel of its own (column / whole-tensor reduction, isolated long row reduction)
    bool needs_store = false;
    int temp = -1;       // temporary buffer index when stored but not an output
    std::vector<uint32_t> consumers;
};

inline bool is_reduce(uint16_t op) { return op >= LT_OP_ROW_SUM && op <= LT_OP_ROW_MIN; }
inline bool is_col_reduce(uint16_t op) { return op >= LT_OP_COL_SUM && op <= LT_OP_COL_MIN; }
inline bool is_all_reduce(uint16_t op) { return op >= LT_OP_ALL_SUM && op <= LT_OP_ALL_MIN; }
inline bool is_shape_op(uint16_t op) { return op >= LT_OP_RESHAPE && op <= LT_OP_UPDATE_SLICE; }
constexpr uint64_t MAX_RESIDENT_COLS = (uint64_t)LT_VM_V * 1024;  // longest row a thread group keeps in registers
inline bool is_factory(uint16_t op) { return op == LT_OP_IOTA || op == LT_OP_PHILOX_BITS; }
inline bool is_float(uint8_t dt) { return dt == LT_F32 || dt == LT_BF16; }

void domain_of(const CNode &n, uint64_t *rows, uint64_t *cols, uint64_t *numel) {
    uint64_t ne = 1;
    for (int i = 0; i < n.rank; ++i) ne *= (uint64_t)n.dims[i];
    uint64_t c = n.rank ? (uint64_t)n.dims[n.rank - 1] : 1;
    *numel = ne;
    *cols = c;
    *rows = c ? ne / c : 0;
}

// class of a value with domain (r, c, ne) inside a group with domain (R, C)
int class_in(uint64_t r, uint64_t c, uint64_t ne, uint64_t R, uint64_t C) {
    if (r == R && c == C) return LT_CLS_FULL;
    if (ne == 1) return LT_CLS_SCALAR;
    if (r == 1 && c == C) return LT_CLS_COLVEC;
    if (c == 1 && r == R) return LT_CLS_ROWVEC;
    return -1;
}

bool approx_sensitive(uint16_t op) {
    switch (op) {
    case LT_OP_DIV: case LT_OP_EXP: case LT_OP_LOG: case LT_OP_TANH: case LT_OP_SQRT: case LT_OP_RSQRT:
    case LT_OP_RECIP: case LT_OP_SIGMOID: case LT_OP_GELU_TANH:
        return true;
    default:
        return false;
    }
}

// does CONVERT from `si` to `so` leave the 32-bit register lanes unchanged?
bool convert_is_alias(int si, int so) {
    if (si == so) return true;
    if (si == LT_BF16 && so == LT_F32) return true;
    if ((si == LT_I32 || si == LT_U32) && (so == LT_I32 || so == LT_U32)) return true;
    if (si == LT_U8 && (so == LT_I32 || so == LT_U32)) return true;
    return false;
}

uint8_t enc_of(int dtype) { return (uint8_t)dtype; }  // ENC_* share lt_dtype numbering for 0..4

// --------------------------------------------------------------------- codegen
struct CodeGen {
    const Canonical &cg;
    std::vector<PNode> &pn;
    Group &g;
    int self;  // index of g
    const std::vector<uint32_t> &emit;  // nodes to compute, topological order
    const std::vector<uint8_t> &in_emit;

    std::vector<int> rep, uses, temp_of, slot_of;
    int temp_val[LT_VM_NT];
    int temp_raw[LT_VM_NT];  // storage dtype still to widen, or -1
    int in_acc = -1;
    int acc_raw = -1;
    bool ok = true;
    bool has_reduce = false, needs_rowcol = false;
    std::vector<uint8_t> tainted;

    CodeGen(const Canonical &cg_, std::vector<PNode> &pn_, Group &g_, int self_, const std::vector<uint32_t> &emit_,
            const std::vector<uint8_t> &in_emit_)
        : cg(cg_), pn(pn_), g(g_), self(self_), emit(emit_), in_emit(in_emit_) {
        size_t n = cg.nodes.size();
        rep.assign(n, -1);
        uses.assign(n, 0);
        temp_of.assign(n, -1);
        slot_of.assign(n, -1);
        tainted.assign(n, 0);
        for (int k = 0; k < LT_VM_NT; ++k) temp_val[k] = -1, temp_raw[k] = -1;
    }

    void emit_ins(uint32_t op, uint32_t imm = 0) {
        LtIns in;
        in.op = op;
        in.imm = imm;
        g.ins.push_back(in);
    }

    // chunk of input v, widened to 32-bit lanes, into register d (0..3 = T0..T3, 4 = ACC); the kernel
    // rewrites the generic opcode into a vector-path one when the pointer allows (see vm.h)
    void emit_load(int d, uint32_t v) { emit_ins(OP_LD + (uint32_t)d, (uint32_t)input_slot(v)); }

    int cls_of(uint32_t v) const {
        const PNode &p = pn[v];
        return class_in(p.rows, p.cols, p.numel, g.rows, g.cols);
    }

    // is v a value this group reads from memory (a device-data leaf or another group's result)?
    bool is_input(uint32_t v) const { return !in_emit[v] && cg.nodes[v].op != N_SCALAR; }

    int input_slot(uint32_t v) {
        if (slot_of[v] >= 0) return slot_of[v];
        const CNode &n = cg.nodes[v];
        IoRef io;
        io.is_store = 0;
        io.dtype = n.dtype;
        io.cls = (uint8_t)cls_of(v);
        io.cnode = v;
        if (n.op == LT_OP_NARROW && pn[v].in_place_slice) {
            // a slice read in place: the parameter it is cut from, an offset, and a row pitch when rows are not contiguous
            const CNode &base = cg.nodes[n.in[0]];
            io.kind = IO_PARAM;
            io.index = (uint32_t)base.param;
            const uint64_t base_cols = (uint64_t)base.dims[base.rank - 1];
            if (n.attr0 == n.rank - 1 && n.rank > 0 && (uint64_t)n.dims[n.rank - 1] != base_cols) {
                io.offset = (uint64_t)n.attr1;
                if (io.cls == LT_CLS_FULL && g.rows > 1) {
                    io.cls = LT_CLS_PITCHED;
                    io.pitch = (uint32_t)base_cols;
                }
            } else {
                uint64_t inner = 1;
                for (int d = 1; d < n.rank; ++d) inner *= (uint64_t)n.dims[d];
                io.offset = (uint64_t)n.attr1 * inner;
            }
        } else if (n.op == N_DEVICE_DATA) {
            io.kind = IO_PARAM;
            io.index = (uint32_t)n.param;
        } else if (n.output >= 0) {
            io.kind = IO_OUTPUT;
            io.index = (uint32_t)n.output;
        } else {
            io.kind = IO_TEMP;
            io.index = 0;  // patched once temporaries are numbered
        }
        if (io.cls == LT_CLS_COLVEC || io.cls == LT_CLS_ROWVEC || io.cls == LT_CLS_PITCHED) needs_rowcol = true;
        slot_of[v] = (int)g.io.size();
        g.io.push_back(io);
        return slot_of[v];
    }

    int imm_slot(const Imm &im, bool dedupe = true) {
        if (dedupe)
            for (size_t i = 0; i < g.imms.size(); ++i)
                if (g.imms[i] == im) return (int)i;
        g.imms.push_back(im);
        return (int)g.imms.size() - 1;
    }

    int scalar_imm(uint32_t v, int dtype) {
        const CNode &n = cg.nodes[v];
        Imm im;
        im.dyn = n.dyn;
        im.sval = n.dyn >= 0 ? 0.0 : n.sval;
        im.enc = enc_of(dtype);
        return imm_slot(im);
    }

    int alloc_temp() {
        for (int k = 0; k < LT_VM_NT; ++k)
            if (temp_val[k] < 0) return k;
        ok = false;
        return 0;
    }

    void drop_if_dead(int v) {
        if (v < 0 || uses[v] > 0) return;
        if (temp_of[v] >= 0) {
            temp_val[temp_of[v]] = -1;
            temp_raw[temp_of[v]] = -1;
            temp_of[v] = -1;
        }
        if (in_acc == v) in_acc = -1;
    }

    // keep the value in ACC alive in a temporary if something still needs it
    void spill_acc(int extra_uses_consumed = 0) {
        if (in_acc < 0) return;
        int v = in_acc;
        if (uses[v] - extra_uses_consumed > 0 && temp_of[v] < 0) {
            int k = alloc_temp();
            if (!ok) return;
            emit_ins((uint16_t)(OP_MOV_T_ACC + k));
            temp_val[k] = v;
            temp_raw[k] = -1;
            temp_of[v] = k;
        }
    }

    static bool needs_widen(int dt) { return dt == LT_BF16 || dt == LT_U8; }

    void widen_temp(int) {}  // loads deliver widened lanes

    // value v available, widened, in a temporary; returns its index
    int ensure_temp(int v) {
        if (temp_of[v] >= 0) {
            widen_temp(temp_of[v]);
            return temp_of[v];
        }
        int k = alloc_temp();
        if (!ok) return 0;
        if (in_acc == v) {
            emit_ins((uint16_t)(OP_MOV_T_ACC + k));
        } else if (is_input((uint32_t)v)) {
            emit_load(k, (uint32_t)v);
        } else {
            ok = false;  // value was never computed: planner bug
            return 0;
        }
        temp_val[k] = v;
        temp_raw[k] = -1;
        temp_of[v] = k;
        return k;
    }

    // value v in ACC (the value currently there is saved first if still needed)
    void ensure_acc(int v) {
        if (in_acc == v) return;
        spill_acc();
        if (!ok) return;
        if (temp_of[v] >= 0) {
            widen_temp(temp_of[v]);
            emit_ins((uint16_t)(OP_MOV_ACC_T + temp_of[v]));
        } else if (is_input((uint32_t)v)) {
            emit_load(LT_VM_NT, (uint32_t)v);
        } else {
            ok = false;
            return;
        }
        in_acc = v;
    }

    void consume(int v) {
        uses[v]--;
    }

    // can v be read straight from memory by the one instruction that uses it?
    bool mem_operand_ok(int v) const { return is_input((uint32_t)v) && uses[v] == 1 && temp_of[v] < 0 && in_acc != v; }

    // Loop-invariant loads: a column vector is the same for every chunk a thread runs (the kernels keep a
    // thread on one column range), so up to `count` of them are loaded once, before the per-chunk body,
    // into temporaries that stay reserved.
    void hoist(int count) {
        int done = 0;
        for (uint32_t n : emit) {
            const CNode &cn = cg.nodes[n];
            for (int i = 0; i < cn.n_in && done < count; ++i) {
                const uint32_t o = (uint32_t)rep_or_self(cn.in[i]);
                if (!is_input(o) || temp_of[o] >= 0 || cls_of(o) != LT_CLS_COLVEC) continue;
                const int k = alloc_temp();
                emit_load(k, o);
                temp_val[k] = (int)o;
                temp_of[o] = k;
                temp_raw[k] = -1;
                uses[o] += 1 << 20;  // never released
                ++done;
            }
        }
        g.n_pro = (uint32_t)g.ins.size();
    }

    int rep_or_self(uint32_t v) const { return rep[v] >= 0 ? rep[v] : (int)v; }

    void count_uses() {
        for (uint32_t n : emit) {
            const CNode &cn = cg.nodes[n];
            for (int i = 0; i < cn.n_in; ++i) uses[cn.in[i]]++;
        }
    }

    void store_result(uint32_t n) {
        // ACC holds node n's value
        const CNode &cn = cg.nodes[n];
        IoRef io;
        io.is_store = 1;
        io.dtype = cn.dtype;
        io.cls = (uint8_t)cls_of(n);
        io.cnode = n;
        if (cn.output >= 0) {
            io.kind = IO_OUTPUT;
            io.index = (uint32_t)cn.output;
        } else {
            io.kind = IO_TEMP;
            io.index = 0;
        }
        if (io.cls == LT_CLS_SCALAR && g.rows == 1) io.cls = LT_CLS_ROWVEC;  // the one value of a one-row group: row 0's
        if (io.cls == LT_CLS_COLVEC || io.cls == LT_CLS_SCALAR) {
            ok = false;  // native members are FULL or ROWVEC by construction
            return;
        }
        if (io.cls == LT_CLS_ROWVEC && !has_reduce) needs_rowcol = true;
        int s = (int)g.io.size();
        g.io.push_back(io);
        emit_ins(OP_ST, (uint32_t)s);
    }

    // ---- one node
    void gen_node(uint32_t n) {
        const CNode &cn = cg.nodes[n];
        const uint16_t op = cn.op;
        const bool store = pn[n].group == self && pn[n].needs_store;
        for (int i = 0; i < cn.n_in; ++i)
            if (tainted[rep_or_self(cn.in[i])] || tainted[cn.in[i]]) tainted[n] = 1;
        if (approx_sensitive(op)) tainted[n] = 1;

        if ((op == LT_OP_CONVERT && convert_is_alias(cg.nodes[cn.in[0]].dtype, cn.dtype)) || op == LT_OP_RESHAPE) {
            int x = rep_or_self(cn.in[0]);
            if (cg.nodes[cn.in[0]].op == N_SCALAR) { ok = false; return; }
            rep[n] = x;
            uses[x] += uses[n] - 1;
            tainted[n] = tainted[x] || tainted[n];
            if (store) {
                ensure_acc(x);
                if (!ok) return;
                store_result(n);
            }
            drop_if_dead(x);
            return;
        }

        int dt = cn.dtype;  // compute dtype of the node
        if (op >= LT_OP_ADD && op <= LT_OP_NE) {
            const bool compare = op >= LT_OP_GT;
            uint32_t xo = cn.in[0], yo = cn.in[1];
            bool xs = cg.nodes[xo].op == N_SCALAR, ys = cg.nodes[yo].op == N_SCALAR;
            int odt = compare ? (xs ? cg.nodes[yo].dtype : cg.nodes[xo].dtype) : dt;  // operand dtype
            int x = xs ? -1 : rep_or_self(xo), y = ys ? -1 : rep_or_self(yo);
            bool swapped = false;
            int src = -1;   // temp index or LT_VM_SRC_S
            uint32_t imm = 0;
            if (xs && ys) {
                spill_acc();
                if (!ok) return;
                emit_ins(OP_MOV_ACC_S, (uint32_t)scalar_imm(xo, odt));
                in_acc = -1;
                src = LT_VM_SRC_S;
                imm = (uint32_t)scalar_imm(yo, odt);
            } else if (ys || xs) {
                int v = ys ? x : y;
                swapped = xs;
                ensure_acc(v);
                if (!ok) return;
                consume(v);
                spill_acc();
                if (!ok) return;
                src = LT_VM_SRC_S;
                imm = (uint32_t)scalar_imm(ys ? yo : xo, odt);
            } else if (x == y) {
                ensure_acc(x);
                if (!ok) return;
                consume(x);
                consume(x);
                if (!compare && is_float((uint8_t)odt) && op == LT_OP_MUL) {
                    spill_acc();
                    if (!ok) return;
                    src = -2;  // square
                } else {
                    src = ensure_temp(x);
                    if (!ok) return;
                }
            } else if (!compare && is_float((uint8_t)dt) && (op == LT_OP_ADD || op == LT_OP_SUB || op == LT_OP_MUL) &&
                       ((mem_operand_ok(y) && (in_acc == x || temp_of[x] < 0)) ||
                        (mem_operand_ok(x) && !mem_operand_ok(y) && (in_acc == y || temp_of[y] < 0)))) {
                // an input read exactly once: fold its load into the arithmetic (memory operand)
                const bool pick_y = mem_operand_ok(y);
                const int mem = pick_y ? y : x, reg = pick_y ? x : y;
                swapped = !pick_y;  // ACC holds the other operand: "ACC (op) mem" must compute x (op) y
                ensure_acc(reg);
                if (!ok) return;
                consume(reg);
                consume(mem);
                spill_acc();
                if (!ok) return;
                const int slot = input_slot((uint32_t)mem);
                const uint32_t k = op == LT_OP_ADD ? F2M_ADD : op == LT_OP_MUL ? F2M_MUL : (swapped ? F2M_RSUB : F2M_SUB);
                emit_ins(OP_F2M + k, (uint32_t)slot);
                src = -3;  // already emitted
            } else {
                // put one operand in ACC (prefer the one already there), the other in a temporary
                if (in_acc == y && in_acc != x) swapped = true;
                else if (in_acc != x) {
                    // neither is in ACC: move the one that is not already in a temporary, or x
                    if (temp_of[x] >= 0 && temp_of[y] < 0) swapped = true;
                }
                int a = swapped ? y : x, b = swapped ? x : y;
                ensure_acc(a);
                if (!ok) return;
                src = ensure_temp(b);
                if (!ok) return;
                consume(a);
                consume(b);
                spill_acc();
                if (!ok) return;
            }
            // opcode
            uint16_t code = 0;
            if (src == -3) {
            } else if (src == -2) {
                code = OP_U_SQUARE;
            } else if (compare) {
                int cc = op - LT_OP_GT;
                if (swapped) { static const int sw[6] = {CC_LT, CC_LE, CC_GT, CC_GE, CC_EQ, CC_NE}; cc = sw[cc]; }
                int ty = is_float((uint8_t)odt) ? 0 : (odt == LT_I32 ? 1 : 2);
                code = (uint16_t)(OP_CMP + (ty * 6 + cc) * LT_VM_NSRC + src);
            } else if (is_float((uint8_t)dt)) {
                int idx;
                switch (op) {
                case LT_OP_ADD: idx = F2_ADD; break;
                case LT_OP_SUB: idx = swapped ? F2_RSUB : F2_SUB; break;
                case LT_OP_MUL: idx = F2_MUL; break;
                case LT_OP_DIV: idx = swapped ? F2_RDIV : F2_DIV; break;
                case LT_OP_MAX: idx = F2_MAX; break;
                default: idx = F2_MIN; break;
                }
                code = (uint16_t)(OP_F2 + idx * LT_VM_NSRC + src);
            } else {
                int idx;
                const bool sgn = dt == LT_I32;
                switch (op) {
                case LT_OP_ADD: idx = I2_ADD; break;
                case LT_OP_SUB: idx = swapped ? I2_RSUB : I2_SUB; break;
                case LT_OP_MUL: idx = I2_MUL; break;
                case LT_OP_MAX: idx = sgn ? I2_MAXS : I2_MAXU; break;
                case LT_OP_MIN: idx = sgn ? I2_MINS : I2_MINU; break;
                case LT_OP_AND: idx = I2_AND; break;
                case LT_OP_OR: idx = I2_OR; break;
                default: idx = I2_XOR; break;
                }
                code = (uint16_t)(OP_I2 + idx * LT_VM_NSRC + src);
            }
            if (src != -3) emit_ins(code, imm);
            if (x >= 0) drop_if_dead(x);
            if (y >= 0) drop_if_dead(y);
        } else if (op == LT_OP_WHERE) {
            uint32_t mo = cn.in[0], ao = cn.in[1], bo = cn.in[2];
            int m = rep_or_self(mo);
            bool as = cg.nodes[ao].op == N_SCALAR, bs = cg.nodes[bo].op == N_SCALAR;
            int a = as ? -1 : rep_or_self(ao), b = bs ? -1 : rep_or_self(bo);
            int mk = ensure_temp(m);
            if (!ok) return;
            bool variant_b = false;  // false: ACC = m ? ACC : src ; true: ACC = m ? src : ACC
            int src;
            uint32_t imm = 0;
            if (as && bs) {
                spill_acc();
                if (!ok) return;
                emit_ins(OP_MOV_ACC_S, (uint32_t)scalar_imm(ao, dt));
                in_acc = -1;
                src = LT_VM_SRC_S;
                imm = (uint32_t)scalar_imm(bo, dt);
            } else if (bs) {
                ensure_acc(a);
                if (!ok) return;
                consume(a);
                spill_acc();
                src = LT_VM_SRC_S;
                imm = (uint32_t)scalar_imm(bo, dt);
            } else if (as) {
                ensure_acc(b);
                if (!ok) return;
                consume(b);
                spill_acc();
                variant_b = true;
                src = LT_VM_SRC_S;
                imm = (uint32_t)scalar_imm(ao, dt);
            } else {
                if (in_acc == b && a != b) variant_b = true;
                int inacc = variant_b ? b : a, other = variant_b ? a : b;
                ensure_acc(inacc);
                if (!ok) return;
                src = ensure_temp(other);
                if (!ok) return;
                consume(inacc);
                consume(other);
                spill_acc();
            }
            if (!ok) return;
            mk = temp_of[m];  // unchanged, but re-read after possible spills
            consume(m);
            emit_ins((uint32_t)((variant_b ? OP_WHERE_B : OP_WHERE_A) + mk * LT_VM_NSRC + src), imm);
            drop_if_dead(m);
            if (a >= 0) drop_if_dead(a);
            if (b >= 0) drop_if_dead(b);
        } else if ((op >= LT_OP_NEG && op <= LT_OP_NOT) || op == LT_OP_CONVERT || is_reduce(op)) {
            uint32_t xo = cn.in[0];
            if (cg.nodes[xo].op == N_SCALAR) {
                spill_acc();
                if (!ok) return;
                emit_ins(OP_MOV_ACC_S, (uint32_t)scalar_imm(xo, cg.nodes[xo].dtype));
                in_acc = -1;
            } else {
                int x = rep_or_self(xo);
                ensure_acc(x);
                if (!ok) return;
                consume(x);
                spill_acc();
                if (!ok) return;
                drop_if_dead(x);
            }
            int si = cg.nodes[xo].dtype;
            if (op == LT_OP_CONVERT) {
                int so = cn.dtype;
                int mid = si == LT_BF16 ? LT_F32 : si;  // registers hold bf16 values as f32
                if (so == LT_F32 || so == LT_BF16) {
                    if (mid == LT_I32) emit_ins(OP_C_I2F);
                    else if (mid == LT_U32 || mid == LT_U8) emit_ins(OP_C_U2F);
                } else if (so == LT_I32) {
                    emit_ins(OP_C_F2I);
                } else if (so == LT_U8) {
                    emit_ins(mid == LT_F32 ? OP_C_NZF : OP_C_NZI);
                }
            } else if (is_reduce(op)) {
                has_reduce = true;
                emit_ins((uint16_t)(OP_RED_SUM + (op - LT_OP_ROW_SUM)));
            } else {
                uint16_t code;
                switch (op) {
                case LT_OP_NEG: code = dt == LT_I32 ? OP_U_INEG : OP_U_NEG; break;
                case LT_OP_ABS: code = dt == LT_I32 ? OP_U_IABS : OP_U_ABS; break;
                case LT_OP_RELU: code = OP_U_RELU; break;
                case LT_OP_EXP: code = OP_U_EXP; break;
                case LT_OP_LOG: code = OP_U_LOG; break;
                case LT_OP_TANH: code = OP_U_TANH; break;
                case LT_OP_SQRT: code = OP_U_SQRT; break;
                case LT_OP_RSQRT: code = OP_U_RSQRT; break;
                case LT_OP_RECIP: code = OP_U_RECIP; break;
                case LT_OP_SQUARE: code = OP_U_SQUARE; break;
                case LT_OP_SIGMOID: code = OP_U_SIGMOID; break;
                case LT_OP_GELU_TANH: code = OP_U_GELU; break;
                default: code = OP_U_NOT; break;
                }
                emit_ins(code);
            }
        } else if (op == LT_OP_IOTA) {
            spill_acc();
            if (!ok) return;
            if ((int)cn.attr0 == cn.rank - 1) {
                emit_ins(OP_IOTA_COL);
                if (g.rows > 1) needs_rowcol = true;
            } else {
                uint64_t inner = 1;
                for (int d = (int)cn.attr0 + 1; d + 1 < cn.rank; ++d) inner *= (uint64_t)cn.dims[d];
                Imm a{-1, (double)inner, ENC_U32}, b{-1, (double)cn.dims[cn.attr0], ENC_U32};
                int s = imm_slot(a, false);
                imm_slot(b, false);
                emit_ins(OP_IOTA_ROW, (uint32_t)s);
                needs_rowcol = true;
            }
        } else if (op == LT_OP_PHILOX_BITS) {
            spill_acc();
            if (!ok) return;
            Imm k0{cn.dyn, 0.0, ENC_LO32}, k1{cn.dyn, 0.0, ENC_HI32}, o0{cn.dyn + 1, 0.0, ENC_LO32}, o1{cn.dyn + 1, 0.0, ENC_HI32};
            int s = imm_slot(k0, false);
            imm_slot(k1, false);
            imm_slot(o0, false);
            imm_slot(o1, false);
            emit_ins(OP_PHILOX, (uint32_t)s);
        } else {
            ok = false;
            return;
        }
        in_acc = (int)n;
        // bf16 nodes: arithmetic happens in f32 and the result is rounded to bf16 (ties to even);
        // a value that is only stored is rounded by the store itself
        if (dt == LT_BF16) {
            bool rounds = (op >= LT_OP_ADD && op <= LT_OP_DIV) || (op >= LT_OP_EXP && op <= LT_OP_GELU_TANH) ||
                          op == LT_OP_ROW_SUM || (op == LT_OP_CONVERT);
            if (rounds && uses[n] > 0) emit_ins(OP_U_RBF16);
        }
        if (store) store_result(n);
        if (uses[n] == 0) in_acc = -1;
    }

    bool run(int hoist_count) {
        count_uses();
        hoist(hoist_count);
        for (uint32_t n : emit) {
            gen_node(n);
            if (!ok) return false;
        }
        if (g.ins.size() > LT_VM_MAX_INS || g.io.size() > LT_VM_MAX_PTR || g.imms.size() > LT_VM_MAX_SCAL) return false;
        return true;
    }
};

// nodes a group must compute: its native members plus the absorbed producers they reach
void emission_list(const Canonical &cg, const std::vector<PNode> &pn, const Group &g, std::vector<uint32_t> &emit,
                   std::vector<uint8_t> &in_emit) {
    emit.clear();
    std::vector<uint32_t> stack(g.members.begin(), g.members.end());
    for (uint32_t m : g.members) in_emit[m] = 1;
    emit = g.members;
    while (!stack.empty()) {
        uint32_t n = stack.back();
        stack.pop_back();
        const CNode &cn = cg.nodes[n];
        for (int i = 0; i < cn.n_in; ++i) {
            uint32_t o = cn.in[i];
            if (pn[o].absorbed && !in_emit[o]) {
                in_emit[o] = 1;
                emit.push_back(o);
                stack.push_back(o);
            }
        }
    }
    std::sort(emit.begin(), emit.end());  // canonical order is topological
}

uint64_t io_bytes(const Group &g, const IoRef &io) {
    uint64_t es = dtype_size(io.dtype);
    switch (io.cls) {
    case LT_CLS_FULL: case LT_CLS_PITCHED: return g.rows * g.cols * es;
    case LT_CLS_COLVEC: return g.cols * es;
    case LT_CLS_ROWVEC: return g.rows * es;
    default: return es;
    }
}

const char *src_name(int s) {
    static const char *n[] = {"T0", "T1", "T2", "T3", "T4"};
    return n[s];
}

std::string disasm(const LtIns &in) {
    char buf[96];
    const int op = in.op;
    auto src_txt = [&](int s) -> std::string {
        if (s == LT_VM_SRC_S) return "S" + std::to_string(in.imm);
        return src_name(s);
    };
    if (op >= OP_MOV_T_ACC && op < OP_MOV_ACC_T) snprintf(buf, sizeof(buf), "T%d = ACC", op - OP_MOV_T_ACC);
    else if (op >= OP_MOV_ACC_T && op < OP_MOV_ACC_S) snprintf(buf, sizeof(buf), "ACC = T%d", op - OP_MOV_ACC_T);
    else if (op == OP_MOV_ACC_S) snprintf(buf, sizeof(buf), "ACC = S%u", in.imm);
    else if (op >= OP_LD && op < OP_LD + LT_VM_ND) {
        if (op - OP_LD < LT_VM_NT) snprintf(buf, sizeof(buf), "T%d = load p%u", op - OP_LD, in.imm);
        else snprintf(buf, sizeof(buf), "ACC = load p%u", in.imm);
    } else if (op >= OP_F2M && op < OP_F2M + F2M_COUNT) {
        static const char *f[] = {"add", "sub", "rsub", "mul"};
        snprintf(buf, sizeof(buf), "ACC = f.%s ACC, load p%u", f[op - OP_F2M], in.imm);
    } else if (op == OP_ST) snprintf(buf, sizeof(buf), "store p%u = ACC", in.imm);
    else if (op == OP_IOTA_COL) snprintf(buf, sizeof(buf), "ACC = iota.col");
    else if (op == OP_IOTA_ROW) snprintf(buf, sizeof(buf), "ACC = iota.row S%u S%u", in.imm, in.imm + 1);
    else if (op == OP_PHILOX) snprintf(buf, sizeof(buf), "ACC = philox S%u..S%u", in.imm, in.imm + 3);
    else if (op >= OP_RED_SUM && op <= OP_RED_MIN) {
        static const char *r[] = {"sum", "max", "min"};
        snprintf(buf, sizeof(buf), "ACC = row_%s ACC", r[op - OP_RED_SUM]);
    } else if (op >= OP_U_NEG && op <= OP_C_NZI) {
        static const char *u[] = {"neg", "abs", "relu", "exp", "log", "tanh", "sqrt", "rsqrt", "recip", "square",
                                  "sigmoid", "gelu_tanh", "round_bf16", "ineg", "iabs", "not", "i2f", "u2f", "f2i",
                                  "nonzero.f", "nonzero.i"};
        snprintf(buf, sizeof(buf), "ACC = %s ACC", u[op - OP_U_NEG]);
    } else if (op >= OP_F2 && op < OP_I2) {
        static const char *f[] = {"add", "sub", "rsub", "mul", "div", "rdiv", "max", "min"};
        int idx = (op - OP_F2) / LT_VM_NSRC, s = (op - OP_F2) % LT_VM_NSRC;
        snprintf(buf, sizeof(buf), "ACC = f.%s ACC, %s", f[idx], src_txt(s).c_str());
    } else if (op >= OP_I2 && op < OP_I2 + I2_COUNT * LT_VM_NSRC) {
        static const char *f[] = {"add", "sub", "rsub", "mul", "and", "or", "xor", "max.s", "min.s", "max.u", "min.u"};
        int idx = (op - OP_I2) / LT_VM_NSRC, s = (op - OP_I2) % LT_VM_NSRC;
        snprintf(buf, sizeof(buf), "ACC = i.%s ACC, %s", f[idx], src_txt(s).c_str());
    } else if (op >= OP_CMP && op < OP_CMP + CMP_COUNT * LT_VM_NSRC) {
        static const char *cc[] = {"gt", "ge", "lt", "le", "eq", "ne"};
        static const char *ty[] = {"f", "s", "u"};
        int idx = (op - OP_CMP) / LT_VM_NSRC, s = (op - OP_CMP) % LT_VM_NSRC;
        snprintf(buf, sizeof(buf), "ACC = cmp.%s.%s ACC, %s", cc[idx % 6], ty[idx / 6], src_txt(s).c_str());
    } else if (op >= OP_WHERE_A && op < OP_WHERE_B) {
        int m = (op - OP_WHERE_A) / LT_VM_NSRC, s = (op - OP_WHERE_A) % LT_VM_NSRC;
        snprintf(buf, sizeof(buf), "ACC = T%d ? ACC : %s", m, src_txt(s).c_str());
    } else if (op >= OP_WHERE_B && op < OP_LIMIT) {
        int m = (op - OP_WHERE_B) / LT_VM_NSRC, s = (op - OP_WHERE_B) % LT_VM_NSRC;
        snprintf(buf, sizeof(buf), "ACC = T%d ? %s : ACC", m, src_txt(s).c_str());
    } else snprintf(buf, sizeof(buf), "op%d", op);
    return buf;
}

}  // namespace

void fastdiv_make(uint32_t d, uint32_t *mul, uint32_t *sh1, uint32_t *sh2) {
    // Division of a 32-bit n by invariant d (Granlund & Montgomery 1994): with l = ceil(log2 d) and
    // m' = floor(2^32 (2^l - d) / d) + 1:  t = mulhi(m', n);  q = (t + ((n - t) >> sh1)) >> sh2.
    uint32_t l = 0;
    while (l < 32 && (1ull << l) < d) ++l;
    uint64_t m = ((1ull << 32) * ((1ull << l) - d)) / d + 1;
    *mul = (uint32_t)m;
    *sh1 = l < 1 ? l : 1;
    *sh2 = l < 1 ? 0 : l - 1;
}

int broadcast_class(const int64_t *dims, int rank, uint64_t rows, uint64_t cols) {
    uint64_t ne = 1;
    for (int i = 0; i < rank; ++i) ne *= (uint64_t)dims[i];
    uint64_t c = rank ? (uint64_t)dims[rank - 1] : 1;
    return class_in(c ? ne / c : 0, c, ne, rows, cols);
}

lt_status build_plan(lt_ctx *c, const Canonical &cg, Plan &plan, bool isolate_long_rows) {
    const size_t N = cg.nodes.size();
    std::vector<PNode> pn(N);
    const bool fuse = c->opt.fusion != 0;

    for (size_t i = 0; i < N; ++i) {
        const CNode &n = cg.nodes[i];
        domain_of(n, &pn[i].rows, &pn[i].cols, &pn[i].numel);
        pn[i].leaf = n.op == N_DEVICE_DATA || n.op == N_SCALAR;
        pn[i].reduce = is_reduce(n.op);
        pn[i].foreign = is_col_reduce(n.op) || is_all_reduce(n.op);
        for (int k = 0; k < n.n_in; ++k) pn[n.in[k]].consumers.push_back((uint32_t)i);
        if (pn[i].numel == 0) return fail(c, LT_ERR_UNSUPPORTED, "empty tensors cannot be part of a flushed graph");
    }

    for (size_t i = 0; i < N; ++i) {
        const CNode &n = cg.nodes[i];
        if (!is_shape_op(n.op)) continue;
        const PNode &src = pn[n.in[0]];
        const bool same_domain = n.op == LT_OP_RESHAPE && src.rows == pn[i].rows && src.cols == pn[i].cols;
        pn[i].foreign = !(same_domain && fuse);
        // A slice of materialised data along the last or the first dimension is a block of rows at a fixed pitch (or one
        // contiguous range): consumers that compute over the slice's own [rows, cols] read it in place.
        if (fuse && n.op == LT_OP_NARROW && cg.nodes[n.in[0]].op == N_DEVICE_DATA && n.output < 0 && !pn[i].consumers.empty() &&
            (n.attr0 == n.rank - 1 || n.attr0 == 0) && src.cols < (1ull << 32)) {
            bool all = true;
            for (uint32_t q : pn[i].consumers) {
                const CNode &qn = cg.nodes[q];
                const bool elementwise = (qn.op >= LT_OP_ADD && qn.op <= LT_OP_NOT) || qn.op == LT_OP_CONVERT || is_reduce(qn.op);
                uint64_t qr = pn[q].rows, qc = pn[q].cols;
                if (is_reduce(qn.op)) qr = pn[i].rows, qc = pn[i].cols;
                if (!elementwise || qr != pn[i].rows || qc != pn[i].cols) all = false;
            }
            if (all) {
                pn[i].in_place_slice = true;
                pn[i].foreign = false;
                pn[i].leaf = true;  // nothing computes it: it is an input like the buffer it points into
            }
        }
    }
    if (isolate_long_rows)
        for (size_t i = 0; i < N; ++i)
            if (pn[i].reduce && pn[cg.nodes[i].in[0]].cols > MAX_RESIDENT_COLS) pn[i].foreign = true;

    // ---- absorbed nodes: cheap producers recomputed inside every consumer group instead of
    // being materialised (index/random factories, and computations on broadcast operands)
    if (fuse) {
        for (size_t i = 0; i < N; ++i) {
            const CNode &n = cg.nodes[i];
            PNode &p = pn[i];
            if (p.leaf || p.reduce || p.foreign || n.output >= 0 || p.consumers.empty()) continue;
            bool okc = true;
            if (is_factory(n.op)) {
                for (uint32_t cidx : p.consumers) {
                    const PNode &q = pn[cidx];
                    uint64_t qr = q.rows, qc = q.cols;
                    if (q.reduce) { qr = p.rows; qc = p.cols; }
                    if (qr != p.rows || qc != p.cols || q.foreign) okc = false;
                }
            } else {
                for (uint32_t cidx : p.consumers) {
                    const PNode &q = pn[cidx];
                    if (q.reduce || q.foreign || q.numel <= p.numel) okc = false;
                }
                for (int k = 0; okc && k < n.n_in; ++k)
                    if (!pn[n.in[k]].leaf && !pn[n.in[k]].absorbed) okc = false;
            }
            p.absorbed = okc;
        }
    }

    // ---- native dependencies of each node (through absorbed producers)
    auto native_deps = [&](uint32_t i, std::vector<uint32_t> &out) {
        out.clear();
        std::vector<uint32_t> stack{(uint32_t)i};
        while (!stack.empty()) {
            uint32_t n = stack.back();
            stack.pop_back();
            const CNode &cn = cg.nodes[n];
            for (int k = 0; k < cn.n_in; ++k) {
                uint32_t o = cn.in[k];
                if (pn[o].leaf) continue;
                if (pn[o].absorbed) stack.push_back(o);
                else out.push_back(o);
            }
        }
    };

    // ---- group assignment
    std::vector<Group> &groups = plan.groups;
    std::vector<uint32_t> deps;
    for (size_t i = 0; i < N; ++i) {
        PNode &p = pn[i];
        if (p.leaf || p.absorbed) continue;
        const CNode &n = cg.nodes[i];
        // the domain the node computes over: a reduction works on its input's rows
        uint64_t dr = p.rows, dc = p.cols;
        if (p.reduce) {
            dr = pn[n.in[0]].rows;
            dc = pn[n.in[0]].cols;
        }
        if (p.foreign && !is_shape_op(n.op)) {
            dr = pn[n.in[0]].rows;
            dc = pn[n.in[0]].cols;
        }
        native_deps((uint32_t)i, deps);
        int gmin = -1;
        for (uint32_t d : deps) gmin = std::max(gmin, pn[d].group);
        int target = -1;
        if (fuse && !p.foreign) {
            auto joinable = [&](int gi) -> bool {
                const Group &g = groups[gi];
                if (g.kind >= K_RED || (int)g.members.size() >= MAX_GROUP_NODES) return false;
                if (g.rows == dr && g.cols == dc) return true;
                // an [R,1] computation on row scalars of a wider group stays with that group
                if (!p.reduce && p.cols == 1 && p.rows == g.rows && g.cols > 1) {
                    for (uint32_t d : deps)
                        if (pn[d].group == gi && pn[d].cols == 1) return true;
                }
                return false;
            };
            if (gmin >= 0 && joinable(gmin)) {
                target = gmin;
                // operands computed in other, older groups of the same domain: pull those groups in,
                // unless a group in between reads them (it would end up before its producer)
                for (uint32_t d : deps) {
                    const int a = pn[d].group;
                    if (a == target || a < 0) continue;
                    Group &ga = groups[a];
                    Group &gb = groups[target];
                    if (ga.kind >= K_RED || ga.rows != gb.rows || ga.cols != gb.cols) continue;
                    if (ga.members.size() + gb.members.size() >= (size_t)MAX_GROUP_NODES) continue;
                    bool legal = true;
                    for (uint32_t m : ga.members) {
                        std::vector<uint32_t> stack{m};
                        while (!stack.empty() && legal) {
                            uint32_t x = stack.back();
                            stack.pop_back();
                            for (uint32_t q : pn[x].consumers) {
                                if (q >= i) continue;  // not placed yet
                                if (pn[q].absorbed) stack.push_back(q);
                                else if (pn[q].group > a && pn[q].group < target) legal = false;
                            }
                        }
                        if (!legal) break;
                    }
                    if (!legal) continue;
                    for (uint32_t m : ga.members) pn[m].group = target;
                    gb.members.insert(gb.members.end(), ga.members.begin(), ga.members.end());
                    std::sort(gb.members.begin(), gb.members.end());
                    ga.members.clear();
                }
            } else if (!p.reduce) {
                // no producer group to join: share a recent group that reads one of the same buffers
                const int lo = std::max(gmin + 1, (int)groups.size() - 8);
                for (int gi = (int)groups.size() - 1; gi >= lo && target < 0; --gi) {
                    const Group &g = groups[gi];
                    if (g.kind >= K_RED || g.rows != dr || g.cols != dc || (int)g.members.size() >= MAX_GROUP_NODES) continue;
                    for (int k = 0; k < n.n_in && target < 0; ++k) {
                        const uint32_t o = n.in[k];
                        if (cg.nodes[o].op != N_DEVICE_DATA) continue;
                        for (uint32_t q : pn[o].consumers)
                            if (q < i && pn[q].group == gi) {
                                target = gi;
                                break;
                            }
                    }
                }
            }
        }
        if (target < 0) {
            groups.emplace_back();
            target = (int)groups.size() - 1;
            groups[target].rows = dr;
            groups[target].cols = dc;
            if (p.foreign && is_shape_op(n.op)) {
                Group &g = groups[target];
                g.kind = K_VIEW;
                g.rows = p.rows;  // the result's own domain
                g.cols = p.cols;
                g.view_op = n.op;
                g.view_a0 = n.attr0;
                g.view_a1 = n.attr1;
                const CNode &src = cg.nodes[n.in[0]];
                g.view_rank = src.rank;
                memcpy(g.view_in_dims, src.dims, sizeof(g.view_in_dims));
                memcpy(g.view_out_dims, n.dims, sizeof(g.view_out_dims));
                if (n.op == LT_OP_UPDATE_SLICE) memcpy(g.view_out_dims, cg.nodes[n.in[1]].dims, sizeof(g.view_out_dims));  // the slice's extent
                if (n.op == LT_OP_RESHAPE) g.view_rank = 1, g.view_in_dims[0] = g.view_out_dims[0] = (int64_t)p.numel;
            } else if (p.foreign) {
                Group &g = groups[target];
                g.kind = K_RED;
                g.red_axis = is_col_reduce(n.op) ? 1 : (is_all_reduce(n.op) ? 2 : 0);
                g.red_kind = (uint8_t)((n.op - LT_OP_ROW_SUM) % 3);
            }
        }
        groups[target].members.push_back((uint32_t)i);
        p.group = target;
    }

    // ---- drop groups emptied by merging
    {
        size_t w = 0;
        for (size_t gi = 0; gi < groups.size(); ++gi) {
            if (groups[gi].members.empty()) continue;
            if (w != gi) groups[w] = std::move(groups[gi]);
            for (uint32_t m : groups[w].members) pn[m].group = (int)w;
            ++w;
        }
        groups.resize(w);
    }

    // ---- code generation (splitting a group that does not fit the machine)
    std::vector<uint8_t> in_emit(N, 0);
    std::vector<uint32_t> emit;
    for (size_t gi = 0; gi < groups.size(); ++gi) {
        for (;;) {
            Group &g = groups[gi];
            // which members must reach memory: outputs, and values read by other groups
            // (recomputed after every split, see below)
            bool done = false;
            emission_list(cg, pn, g, emit, in_emit);
            for (uint32_t m : g.members) {
                PNode &p = pn[m];
                p.needs_store = cg.nodes[m].output >= 0;
            }
            // consumers in other groups (through absorbed chains)
            for (uint32_t m : g.members) {
                std::vector<uint32_t> stack{m};
                while (!stack.empty() && !pn[m].needs_store) {
                    uint32_t n = stack.back();
                    stack.pop_back();
                    for (uint32_t q : pn[n].consumers) {
                        if (pn[q].absorbed) stack.push_back(q);
                        else if (pn[q].group != (int)gi) pn[m].needs_store = true;
                    }
                }
            }
            if (g.kind == K_VIEW) {
                // a copy kernel: the inputs in order, then the result; all dense buffers
                const uint32_t m = g.members[0];
                pn[m].needs_store = true;
                g.ins.clear();
                g.io.clear();
                g.imms.clear();
                auto slot_for = [&](uint32_t v, bool store) {
                    const CNode &vn = cg.nodes[v];
                    IoRef io;
                    io.is_store = store ? 1 : 0;
                    io.dtype = vn.dtype;
                    io.cls = LT_CLS_FULL;
                    io.cnode = v;
                    if (vn.op == N_DEVICE_DATA) io.kind = IO_PARAM, io.index = (uint32_t)vn.param;
                    else if (vn.output >= 0) io.kind = IO_OUTPUT, io.index = (uint32_t)vn.output;
                    else io.kind = IO_TEMP, io.index = 0;
                    g.io.push_back(io);
                };
                for (int k = 0; k < cg.nodes[m].n_in; ++k) slot_for(cg.nodes[m].in[k], false);
                slot_for(m, true);
                g.flavour = 1;
                for (uint32_t nn : emit) in_emit[nn] = 0;
                break;
            }
            if (g.kind == K_RED) {
                // a kernel of its own: slot 0 = the input, slot 1 = the result; no register program
                const uint32_t m = g.members[0];
                const uint32_t src = cg.nodes[m].in[0];
                pn[m].needs_store = true;
                g.ins.clear();
                g.io.clear();
                g.imms.clear();
                auto slot_for = [&](uint32_t v, bool store) {
                    const CNode &vn = cg.nodes[v];
                    IoRef io;
                    io.is_store = store ? 1 : 0;
                    io.dtype = vn.dtype;
                    io.cls = store ? (uint8_t)(g.red_axis == 0 ? LT_CLS_ROWVEC : g.red_axis == 1 ? LT_CLS_COLVEC : LT_CLS_SCALAR) : (uint8_t)LT_CLS_FULL;
                    io.cnode = v;
                    if (vn.op == N_DEVICE_DATA) io.kind = IO_PARAM, io.index = (uint32_t)vn.param;
                    else if (vn.output >= 0) io.kind = IO_OUTPUT, io.index = (uint32_t)vn.output;
                    else io.kind = IO_TEMP, io.index = 0;
                    g.io.push_back(io);
                };
                slot_for(src, false);
                slot_for(m, true);
                g.flavour = 1;
                for (uint32_t nn : emit) in_emit[nn] = 0;
                break;
            }
            int n_inputs = 0;
            {
                std::vector<uint32_t> seen;
                for (uint32_t n : emit) {
                    const CNode &cn = cg.nodes[n];
                    for (int k = 0; k < cn.n_in; ++k) {
                        uint32_t o = cn.in[k];
                        if (!in_emit[o] && cg.nodes[o].op != N_SCALAR && std::find(seen.begin(), seen.end(), o) == seen.end())
                            seen.push_back(o);
                    }
                }
                n_inputs = (int)seen.size();
            }
            (void)n_inputs;  // loads are issued where first needed: staged inputs are already on chip
            for (int pre = (g.rows > 1 ? LT_VM_NT - 1 : 0); pre >= 0 && !done; --pre) {
                g.ins.clear();
                g.io.clear();
                g.imms.clear();
                CodeGen cgen(cg, pn, g, (int)gi, emit, in_emit);
                if (cgen.run(pre)) {
                    done = true;
                    g.kind = cgen.has_reduce ? K_ROW : K_EW;
                    g.rowcol = cgen.needs_rowcol;
                    bool fast = c->opt.fast_math != 0;
                    bool any_store = false;
                    for (const IoRef &io : g.io) {
                        if (!io.is_store) continue;
                        any_store = true;
                        if (io.dtype == LT_F32) fast = false;
                        else if (io.dtype != LT_BF16 && cgen.tainted[io.cnode]) fast = false;
                    }
                    g.flavour = (fast && any_store) ? 0 : (c->opt.ieee ? 2 : 1);
                }
            }
            for (uint32_t n : emit) in_emit[n] = 0;
            if (done) break;
            if (g.members.size() <= 1) return fail(c, LT_ERR_UNSUPPORTED, "an operation does not fit the register program limits");
            // split: the later half of the members moves to a new group right after this one
            size_t half = g.members.size() / 2;
            Group tail;
            tail.rows = g.rows;
            tail.cols = g.cols;
            tail.members.assign(g.members.begin() + half, g.members.end());
            g.members.resize(half);
            groups.insert(groups.begin() + gi + 1, std::move(tail));
            for (size_t k = gi + 1; k < groups.size(); ++k)
                for (uint32_t m : groups[k].members) pn[m].group = (int)k;
            // a row-scalar member that lost its reduction partner keeps the group's domain; fine
        }
    }

    // ---- number temporaries and patch the slots that refer to them
    for (size_t gi = 0; gi < groups.size(); ++gi) {
        Group &g = groups[gi];
        for (IoRef &io : g.io) {
            if (io.kind != IO_TEMP) continue;
            PNode &p = pn[io.cnode];
            if (p.temp < 0) {
                p.temp = (int)plan.temp_bytes.size();
                plan.temp_bytes.push_back((size_t)p.numel * dtype_size(cg.nodes[io.cnode].dtype));
            }
            io.index = (uint32_t)p.temp;
        }
        g.bytes = 0;
        for (const IoRef &io : g.io) g.bytes += io_bytes(g, io);
        if (g.kind == K_VIEW) {
            g.bytes = 0;
            for (const IoRef &io : g.io) g.bytes += pn[io.cnode].numel * dtype_size(io.dtype);
        }
        if (g.kind == K_RED) {
            const size_t scratch = lt_reduce_scratch_bytes(g.red_axis, g.rows, g.cols, c->sm_count);
            if (scratch) {
                g.scratch_temp = (int32_t)plan.temp_bytes.size();
                plan.temp_bytes.push_back(scratch);
            }
        }
        g.long_row = g.kind == K_ROW && g.cols > MAX_RESIDENT_COLS;
        if (g.long_row && g.cols >= (1ull << 28)) return fail(c, LT_ERR_UNSUPPORTED, "rows of a fused reduction are limited to 2^28 elements");
        if (g.kind == K_EW && g.rowcol) {
            uint64_t cpr = (g.cols + LT_VM_V - 1) / LT_VM_V;
            if (g.rows * cpr >= (1ull << 31) || g.rows >= (1ull << 31) || g.cols >= (1ull << 31))
                return fail(c, LT_ERR_UNSUPPORTED, "broadcast group too large for 32-bit chunk indexing");
        }
        if (g.kind == K_ROW && g.rows >= (1ull << 32)) return fail(c, LT_ERR_UNSUPPORTED, "too many rows");
        if (g.kind == K_EW && !g.rowcol && (g.rows * g.cols + LT_VM_V - 1) / LT_VM_V >= (1ull << 31))
            return fail(c, LT_ERR_UNSUPPORTED, "tensor too large for 32-bit chunk indexing");
    }

    // ---- a column or whole-tensor reduction whose input is computed by an elementwise group for it alone: the first
    // stage moves into that group (its kernel reduces the value instead of storing it, lt_c_ewred), the reduction
    // group keeps the second stage.  The input is never materialised.  Only kernels built for the program can do
    // this; the split variant of the plan is the graph without it.
    if (fuse && !isolate_long_rows && c->opt.compiled) {
        for (size_t g2i = 0; g2i < groups.size(); ++g2i) {
            Group &g2 = groups[g2i];
            if (g2.kind != K_RED || g2.red_axis == 0 || g2.scratch_temp < 0 || g2.io.size() != 2 || g2.io[0].kind != IO_TEMP) continue;
            const uint32_t v = g2.io[0].cnode;
            const int g1i = pn[v].group;
            if (g1i < 0 || (size_t)g1i >= g2i) continue;
            Group &g1 = groups[g1i];
            if (g1.kind != K_EW || g1.rows != g2.rows || g1.cols != g2.cols) continue;
            if (g1.fused_red) {  // a group may reduce up to three values, all over the same axis
                size_t have = 0;
                for (const IoRef &io : g1.io) have += io.cls >= LT_CLS_REDUCED ? 1 : 0;
                if (g1.red_axis != g2.red_axis || have >= 3) continue;
            }
            if (g2.rows >= (1ull << 31) || g2.cols >= (1ull << 31)) continue;
            const bool whole_chunks = (g1.rowcol || g2.red_axis == 1) ? (g1.cols % LT_VM_V) == 0 : ((g1.rows * g1.cols) % LT_VM_V) == 0;
            if (!whole_chunks) continue;
            size_t readers = 0;
            for (const Group &g : groups)
                for (const IoRef &io : g.io)
                    if (!io.is_store && io.kind == IO_TEMP && io.cnode == v) ++readers;
            int st = -1;
            for (size_t q = 0; q < g1.io.size(); ++q)
                if (g1.io[q].is_store && g1.io[q].kind == IO_TEMP && g1.io[q].cnode == v && g1.io[q].cls == LT_CLS_FULL) st = (int)q;
            if (readers != 1 || st < 0) continue;
            plan.temp_bytes[pn[v].temp] = 0;  // nothing is written there any more
            IoRef &out = g1.io[st];
            out.cls = (uint8_t)(LT_CLS_REDUCED + 3 * (g2.red_axis - 1) + g2.red_kind);
            out.index = (uint32_t)g2.scratch_temp;
            g1.fused_red = true;
            g1.red_axis = g2.red_axis;
            if (g2.red_axis == 1) g1.rowcol = true;  // the kernel walks rows and columns
            g2.from_partials = true;
            g2.io[0].index = (uint32_t)g2.scratch_temp;
            g1.bytes -= g1.rows * g1.cols * dtype_size(out.dtype);
            g2.bytes = 0;
        }
    }

    // ---- outputs
    plan.n_params = (uint32_t)cg.param_node.size();
    plan.n_dyn = (uint32_t)cg.dyn.size();
    plan.outputs.resize(cg.outputs.size());
    for (size_t k = 0; k < cg.outputs.size(); ++k) {
        const CNode &n = cg.nodes[cg.outputs[k]];
        OutputPlan &o = plan.outputs[k];
        o.dtype = n.dtype;
        o.rank = n.rank;
        memcpy(o.dims, n.dims, sizeof(o.dims));
        o.bytes = (size_t)pn[cg.outputs[k]].numel * dtype_size(n.dtype);
        o.donated_param = -1;
    }

    // ---- launches: bundle isomorphic independent flat groups (horizontal fusion)
    std::vector<int> launch_of(groups.size(), -1);
    {
        // outputs that some group loads: their producers cannot move
        std::vector<uint8_t> output_loaded(cg.outputs.size(), 0);
        for (const Group &g : groups)
            for (const IoRef &io : g.io)
                if (!io.is_store && io.kind == IO_OUTPUT) output_loaded[io.index] = 1;
        std::map<std::string, std::vector<uint32_t>> buckets;
        std::vector<std::string> sig(groups.size());
        if (fuse && c->opt.horizontal) {
            for (size_t gi = 0; gi < groups.size(); ++gi) {
                const Group &g = groups[gi];
                bool el = g.kind == K_EW && !g.rowcol && g.ins.size() <= LT_MULTI_MAX_INS && g.io.size() <= LT_MULTI_MAX_SLOTS &&
                          g.rows * g.cols < (1ull << 32);
                for (const IoRef &io : g.io) {
                    if (io.cls != LT_CLS_FULL) el = false;
                    if (io.is_store ? (io.kind != IO_OUTPUT || output_loaded[io.index]) : io.kind != IO_PARAM) el = false;
                }
                if (!el) continue;
                std::string s;
                s.push_back((char)('0' + g.flavour));
                s.append((const char *)g.ins.data(), g.ins.size() * sizeof(LtIns));
                for (const Imm &im : g.imms) {
                    s.append((const char *)&im.dyn, sizeof(im.dyn));
                    s.append((const char *)&im.sval, sizeof(im.sval));
                    s.push_back((char)im.enc);
                }
                for (const IoRef &io : g.io) {
                    s.push_back((char)io.dtype);
                    s.push_back((char)io.is_store);
                }
                sig[gi] = s;
                buckets[s].push_back((uint32_t)gi);
            }
        }
        for (size_t gi = 0; gi < groups.size(); ++gi) {
            if (launch_of[gi] >= 0) continue;
            const Group &g = groups[gi];
            auto it = sig[gi].empty() ? buckets.end() : buckets.find(sig[gi]);
            if (it != buckets.end() && it->second.size() >= 2) {
                const std::vector<uint32_t> &all = it->second;
                size_t pos = 0;
                const size_t slots = g.io.size();
                const size_t per = std::min<size_t>(LT_MULTI_MAX_INST, LT_MULTI_MAX_PTRS / std::max<size_t>(slots, 1));
                while (pos < all.size()) {
                    Launch L;
                    L.kind = K_MULTI;
                    L.flavour = g.flavour;
                    size_t cnt = std::min(per, all.size() - pos);
                    for (size_t k = 0; k < cnt; ++k) {
                        L.groups.push_back(all[pos + k]);
                        launch_of[all[pos + k]] = (int)plan.launches.size();
                        L.bytes += groups[all[pos + k]].bytes;
                    }
                    pos += cnt;
                    plan.launches.push_back(std::move(L));
                }
            } else {
                Launch L;
                L.kind = g.kind;
                L.flavour = g.flavour;
                L.groups.push_back((uint32_t)gi);
                L.bytes = g.bytes;
                launch_of[gi] = (int)plan.launches.size();
                plan.launches.push_back(std::move(L));
            }
        }
    }

    // ---- donation (Section 4.3): write an output into the parameter buffer its tensor used to
    // name when every read of that buffer is by the writing program itself, at the same element
    // and before the store, or by an earlier launch
    {
        std::vector<std::vector<std::pair<uint32_t, uint32_t>>> readers(plan.n_params);  // (group, slot)
        for (size_t gi = 0; gi < groups.size(); ++gi)
            for (size_t s = 0; s < groups[gi].io.size(); ++s) {
                const IoRef &io = groups[gi].io[s];
                if (!io.is_store && io.kind == IO_PARAM) readers[io.index].push_back({(uint32_t)gi, (uint32_t)s});
            }
        for (size_t gi = 0; gi < groups.size(); ++gi) {
            Group &g = groups[gi];
            for (size_t s = 0; s < g.io.size(); ++s) {
                const IoRef &st = g.io[s];
                if (!st.is_store || st.kind != IO_OUTPUT) continue;
                int32_t p = cg.donor_param[st.index];
                if (p < 0 || st.cls != LT_CLS_FULL) continue;
                bool safe = true;
                for (auto &rd : readers[p]) {
                    const uint32_t rg = rd.first;
                    if (rg == gi && g.kind == K_VIEW) {
                        // update_slice rewrites only the slice of its base: in place when the base (slot 0) is the one
                        // read of the buffer; the other shape operations move every element
                        if (g.view_op != LT_OP_UPDATE_SLICE || rd.second != 0) { safe = false; break; }
                    } else if (rg == gi) {
                        const IoRef &ld = groups[rg].io[rd.second];
                        if (ld.cls != LT_CLS_FULL || ld.offset != 0) { safe = false; break; }  // (a slice reads other elements than the store's)
                        // the load must come before the store in program order
                        int ld_pos = -1, st_pos = -1;
                        for (size_t q = 0; q < g.ins.size(); ++q) {
                            const LtIns &in = g.ins[q];
                            const bool loads = (in.op >= OP_LD && in.op < OP_LD + LT_VM_ND) || (in.op >= OP_F2M && in.op < OP_F2M + F2M_COUNT);
                            if (loads && in.imm == rd.second && ld_pos < 0) ld_pos = (int)q;
                            if (in.op == OP_ST && in.imm == s) st_pos = (int)q;
                        }
                        if (ld_pos < 0 || st_pos < 0 || ld_pos > st_pos) { safe = false; break; }
                    } else if (launch_of[rg] >= launch_of[gi]) {
                        safe = false;
                        break;
                    }
                }
                if (safe) plan.outputs[st.index].donated_param = p;
            }
        }
    }

    // ---- parameter blocks: everything that does not change between hits is filled in now
    for (Launch &L : plan.launches) {
        if (L.kind == K_MULTI) {
            L.mp.reset(new LtMultiParams());
            LtMultiParams &P = *L.mp;
            memset(&P, 0, sizeof(P));
            const Group &g0 = groups[L.groups[0]];
            P.n_ins = (uint32_t)g0.ins.size();
            memcpy(P.ins, g0.ins.data(), g0.ins.size() * sizeof(LtIns));
            P.n_slots = (uint32_t)g0.io.size();
            for (size_t s = 0; s < g0.io.size(); ++s) P.io_dtype[s] = g0.io[s].dtype;
            P.n_inst = (uint32_t)L.groups.size();
            const uint32_t per_super = LT_EW_THREADS * LT_MULTI_SUB * LT_VM_V;
            uint32_t acc = 0;
            for (size_t k = 0; k < L.groups.size(); ++k) {
                const Group &g = groups[L.groups[k]];
                uint32_t ne = (uint32_t)(g.rows * g.cols);
                P.super_prefix[k] = acc;
                P.numel[k] = ne;
                acc += (ne + per_super - 1) / per_super;
            }
            P.super_prefix[L.groups.size()] = acc;
            P.total_super = acc;
        } else if (L.kind < K_RED) {
            L.kp.reset(new LtKParams());
            LtKParams &P = *L.kp;
            memset(&P, 0, sizeof(P));
            const Group &g = groups[L.groups[0]];
            P.n_ins = (uint32_t)g.ins.size();
            P.n_pro = g.n_pro;
            memcpy(P.ins, g.ins.data(), g.ins.size() * sizeof(LtIns));
            for (size_t s = 0; s < g.io.size(); ++s) {
                P.io_dtype[s] = g.io[s].dtype;
                P.io_class[s] = g.io[s].cls;
                P.pitch[s] = g.io[s].pitch;
            }
            P.n = g.rows * g.cols;
            P.rowcol = g.rowcol ? 1u : 0u;
            P.rows = (uint32_t)g.rows;
            P.cols = (uint32_t)g.cols;
            P.cpr = (uint32_t)((g.cols + LT_VM_V - 1) / LT_VM_V);
            fastdiv_make(P.cpr ? P.cpr : 1, &P.div_mul, &P.div_sh1, &P.div_sh2);
            P.n_chunks = g.rowcol ? (uint64_t)g.rows * P.cpr : (P.n + LT_VM_V - 1) / LT_VM_V;
            if (g.kind == K_ROW && !g.long_row) {
                uint32_t grp = 1, lg = 0;
                while (grp < P.cpr) grp <<= 1, ++lg;
                P.group = grp;
                P.group_log2 = lg;
                L.threads = grp > 256 ? grp : 256;
                P.rows_per_cta = L.threads / grp;
            }
        }
    }
    // ---- ahead-of-time compiled kernels: exact lookup of each launch's program
    bool unfused_long_row = false;
    for (Launch &L : plan.launches) {
        const Group &g = groups[L.groups[0]];
        if (L.kind >= K_RED) continue;
        uint8_t dt[LT_VM_MAX_PTR] = {0}, cl[LT_VM_MAX_PTR] = {0};
        for (size_t s = 0; s < g.io.size() && s < LT_VM_MAX_PTR; ++s) {
            dt[s] = g.io[s].dtype;
            cl[s] = L.kind == K_MULTI ? (uint8_t)LT_CLS_FULL : g.io[s].cls;
        }
        L.compiled = c->opt.ignore_table ? -1 : lt_compiled_find(L.kind, L.flavour, g.ins.data(), (uint32_t)g.ins.size(), g.n_pro, dt, cl, (uint32_t)g.io.size());
        if (L.compiled < 0 && c->opt.compiled && c->opt.specialise && jit_available()) {
            // no table entry: describe the program for the run-time specialiser
            std::unique_ptr<JitProgram> jp(new JitProgram());
            jp->kind = L.kind;
            jp->flavour = L.flavour;
            jp->n_pro = g.n_pro;
            jp->ins = g.ins;
            jp->dtype.assign(dt, dt + g.io.size());
            jp->cls.assign(cl, cl + g.io.size());
            jp->long_row = g.long_row;
            if (L.kind == K_ROW && !g.long_row) {
                const uint32_t cpr = (uint32_t)((g.cols + LT_VM_V - 1) / LT_VM_V);
                bool four_byte = false;
                for (const IoRef &io : g.io)
                    if (!io.is_store && io.cls == LT_CLS_FULL && dtype_size(io.dtype) == 4) four_byte = true;
                jp->row_u = row_chunks_per_thread(cpr, g.n_pro > 0 && !jit_integer_heavy(*jp), four_byte);  // (the executor's choice)
            }
            if (L.kind == K_ROW && g.long_row) {
                unsigned k = 0;
                int u = 0;
                if (cluster_shape((uint32_t)((g.cols + LT_VM_V - 1) / LT_VM_V), g.n_pro > 0, c->opt.cluster, c->opt.compiled_row_u, &k, &u)) jp->cluster_u = u;
            }
            if (jit_supported(*jp)) L.jit_program = std::move(jp);
            // a long-row group is only worth keeping fused if its kernel is there when the flush runs
            if (L.jit_program && (g.long_row || g.fused_red) && c->opt.specialise == 1) {
                L.jit = jit_request(*L.jit_program, true);
                if (!L.jit || L.jit->state.load() != 1) L.jit_failed = true;
            }
        }
        // (in the background mode the group stays fused: until its kernel has been built the executor runs the plan's
        // split variant instead, as it does when a fused launch meets unaligned pointers)
        const bool long_ok = L.compiled >= 0 || (L.jit && !L.jit_failed) || (L.jit_program && c->opt.specialise == 2 && c->device != LT_DEVICE_NONE);
        if ((g.long_row || g.fused_red) && (!long_ok || !c->opt.compiled)) unfused_long_row = true;
    }
    if (unfused_long_row) {
        // Only the kernels instantiated at build time walk a long row in slices.  A long-row group without one is
        // planned again with each of its reductions as a kernel of its own; what surrounds them becomes elementwise
        // groups that read the reductions' results as one value per row.
        if (isolate_long_rows) return fail(c, LT_ERR_UNSUPPORTED, "a long-row group could not be planned");
        plan.groups.clear();
        plan.launches.clear();
        plan.temp_bytes.clear();
        plan.outputs.clear();
        return build_plan(c, cg, plan, true);
    }
    return LT_OK;
}

std::string describe_plan(const Plan &plan) {
    std::string s;
    char buf[256];
    snprintf(buf, sizeof(buf), "plan: %zu launches, %zu groups, %u params, %u runtime slots, %zu outputs, %zu temporaries\n",
             plan.launches.size(), plan.groups.size(), plan.n_params, plan.n_dyn, plan.outputs.size(), plan.temp_bytes.size());
    s += buf;
    for (size_t k = 0; k < plan.outputs.size(); ++k)
        if (plan.outputs[k].donated_param >= 0) {
            snprintf(buf, sizeof(buf), "  output %zu donated param %d\n", k, plan.outputs[k].donated_param);
            s += buf;
        }
    static const char *kind[] = {"elementwise", "row", "multi", "reduce", "view"};
    static const char *cls[] = {"full", "colvec", "rowvec", "scalar", "pitched"};
    static const char *reduced[] = {"reduced-over-rows(sum)", "reduced-over-rows(max)", "reduced-over-rows(min)",
                                    "reduced-over-all(sum)",  "reduced-over-all(max)",  "reduced-over-all(min)"};
    static const char *iok[] = {"param", "output", "temp"};
    for (size_t li = 0; li < plan.launches.size(); ++li) {
        const Launch &L = plan.launches[li];
        const Group &g = plan.groups[L.groups[0]];
        snprintf(buf, sizeof(buf), "launch %zu: %s %s instances=%zu rows=%llu cols=%llu %s bytes=%llu\n", li, kind[L.kind],
                 L.flavour == 0 ? "fast" : (L.flavour == 1 ? "precise" : "ieee"), L.groups.size(), (unsigned long long)g.rows, (unsigned long long)g.cols,
                 g.rowcol ? "rowcol" : "flat", (unsigned long long)L.bytes);
        s += buf;
        if (L.kind == K_VIEW) {
            snprintf(buf, sizeof(buf), "  copy kernel: %s\n", op_name(g.view_op));
            s += buf;
        } else if (L.kind == K_RED) {
            static const char *axis[] = {"rows", "columns", "all"}, *what[] = {"sum", "max", "min"};
            snprintf(buf, sizeof(buf), "  reduction kernel: %s over %s%s\n", what[g.red_kind], axis[g.red_axis],
                     g.from_partials ? ", second stage only (the first is in the kernel that computes the input)" : g.scratch_temp >= 0 ? ", two stages" : "");
            s += buf;
        } else {
            // the exact identity of the program: what the table of compiled programs is keyed on
            std::string key = "  key: " + std::to_string(L.kind) + " " + std::to_string(L.flavour) + " " + std::to_string(g.n_pro) + " |";
            for (const IoRef &io : g.io) key += " " + std::to_string(io.dtype);
            key += " |";
            for (const IoRef &io : g.io) key += " " + std::to_string(L.kind == K_MULTI ? 0 : io.cls);
            key += " |";
            for (const LtIns &in : g.ins) key += " " + std::to_string(in.op) + ":" + std::to_string(in.imm);
            s += key + "\n";
            s += std::string("  compiled: ") + (L.compiled >= 0 ? lt_compiled_name(L.compiled) : "no") + "\n";
            if (L.jit_program) {
                const int st = L.jit ? L.jit->state.load() : 2;
                s += std::string("  specialised at run time: ") + (L.jit_failed || st < 0 ? "failed" : st == 1 ? "ready" : st == 0 ? "being compiled" : "not requested yet") + "\n";
            }
        }
        for (size_t q = 0; q < g.io.size(); ++q) {
            const IoRef &io = g.io[q];
            snprintf(buf, sizeof(buf), "  p%zu: %s %s %s %s%u\n", q, io.is_store ? "store" : "load", dtype_name(io.dtype),
                     io.cls >= LT_CLS_REDUCED ? reduced[io.cls - LT_CLS_REDUCED] : cls[io.cls], iok[io.kind], io.index);
            s += buf;
        }
        for (size_t q = 0; q < g.imms.size(); ++q) {
            const Imm &im = g.imms[q];
            if (im.dyn >= 0) snprintf(buf, sizeof(buf), "  S%zu: runtime slot %d enc %d\n", q, im.dyn, im.enc);
            else snprintf(buf, sizeof(buf), "  S%zu: const %g enc %d\n", q, im.sval, im.enc);
            s += buf;
        }
        for (size_t q = 0; q < g.ins.size(); ++q) {
            if (q == g.n_pro && g.n_pro) s += "       -- per chunk:\n";
            snprintf(buf, sizeof(buf), "  %3zu  ", q);
            s += buf;
            s += disasm(g.ins[q]);
            s += "\n";
        }
    }
    if (plan.split) s += "-- the same graph with long row reductions as kernels of their own (used when the fused kernel cannot run):\n" + describe_plan(*plan.split);
    return s;
}

}  // namespace lt
