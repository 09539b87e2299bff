// Recorder, liveness arena and the C ABI (lazytensor.h).
#include "compiled.h"
#include "engine.h"
#include "launch.h"

#include <atomic>
#include <chrono>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <algorithm>

using namespace lt;

namespace {

std::atomic<uint32_t> g_next_tag{1};

inline uint64_t now_ns() {
    return (uint64_t)std::chrono::duration_cast<std::chrono::nanoseconds>(
               std::chrono::steady_clock::now().time_since_epoch())
        .count();
}

// Host-time accounting of lt_stats.  The per-call cost matters: lt_op is timed, and recording a node takes little
// more than a hundred nanoseconds.  On x86-64 the time-stamp counter is read (a few nanoseconds) and the ticks are
// scaled to nanoseconds when the statistics are read; elsewhere the steady clock is used directly.
#if defined(__x86_64__)
inline uint64_t ticks_now() { return __builtin_ia32_rdtsc(); }
const uint64_t g_tick0 = ticks_now(), g_ns0 = now_ns();
inline double ns_per_tick() {
    const uint64_t dt = ticks_now() - g_tick0, dn = now_ns() - g_ns0;
    return dt && dn > 1000000 ? (double)dn / (double)dt : 0.4;  // (before a millisecond has passed: a nominal 2.5 GHz)
}
#else
inline uint64_t ticks_now() { return now_ns(); }
inline double ns_per_tick() { return 1.0; }
#endif

// The recording calls are far more frequent than anything else and, once a trace is only matched, cost about as much
// as two reads of the counter: one call in eight is timed and counted eight times.
struct RecordTimer {
    lt_ctx *c;
    uint64_t t0;
    explicit RecordTimer(lt_ctx *ctx) : c(ctx), t0((++ctx->record_calls & 7u) ? 0 : ticks_now()) {}
    ~RecordTimer() {
        if (t0) c->stats.ns_record += 8 * (ticks_now() - t0);
    }
};

struct Timer {
    uint64_t &acc;
    uint64_t t0;
    explicit Timer(uint64_t &a) : acc(a), t0(ticks_now()) {}
    ~Timer() { acc += ticks_now() - t0; }
};

inline lt_tensor make_handle(const lt_ctx *c, uint32_t slot) {
    return ((uint64_t)c->tag << 48) | ((uint64_t)(c->tensors[slot].gen & 0xffffu) << 32) | (uint64_t)(slot + 1);
}

lt_status sync_view_of(lt_ctx *c, uint32_t slot);
void trace_materialise(lt_ctx *c);

// Every entry point that looks at a tensor's computation resolves its handles here.  A trace that has so far only
// been matched against the previous one (its tensors have no IR yet) is first turned into the real thing.
lt_status lookup(lt_ctx *c, lt_tensor h, uint32_t *slot) {
    if (c->trace.mode == TM_MATCH && c->trace.cursor) trace_materialise(c);
    if ((uint16_t)(h >> 48) != c->tag) return fail(c, LT_ERR_DEVICE, "tensor handle belongs to another context");
    uint32_t s = (uint32_t)(h & 0xffffffffu);
    if (s == 0 || s > c->tensors.size()) return fail(c, LT_ERR_INVALID_ARG, "unknown tensor handle");
    s -= 1;
    const TensorRec &t = c->tensors[s];
    if (!t.live || (t.gen & 0xffffu) != (uint32_t)((h >> 32) & 0xffffu))
        return fail(c, LT_ERR_INVALID_ARG, "tensor handle was released");
    *slot = s;
    if (t.view_base != NONE) return sync_view_of(c, s);  // a view first catches up with its base
    return LT_OK;
}

uint32_t tensor_new(lt_ctx *c, uint32_t node) {
    uint32_t slot;
    if (c->trace.force_slot != NONE) {
        // the tensor exists already as a handle without IR (trace matching): it now gets its node
        slot = c->trace.force_slot;
        c->trace.force_slot = NONE;
        TensorRec &t = c->tensors[slot];
        t.node = node;
        t.vflags = 0;
        node_ref(c, node);
        c->nodes[node].tensor_refs++;
        return slot;
    }
    if (!c->free_tensors.empty()) {
        slot = c->free_tensors.back();
        c->free_tensors.pop_back();
    } else {
        slot = (uint32_t)c->tensors.size();
        c->tensors.emplace_back();
    }
    TensorRec &t = c->tensors[slot];
    t.node = node;
    t.gen += 1;
    t.donor = NONE;
    t.seq = c->next_seq++;
    t.live = true;
    t.queued = false;
    t.view_base = NONE;
    t.view_op = 0;
    t.version = 0;
    t.base_seen = 0;
    t.vflags = 0;
    node_ref(c, node);
    c->nodes[node].tensor_refs++;
    return slot;
}

inline bool is_leaf(const Node &n) { return n.op == N_DEVICE_DATA || n.op == N_SCALAR; }

void queue_pending(lt_ctx *c, uint32_t slot) {
    TensorRec &t = c->tensors[slot];
    if (!t.queued) {
        t.queued = true;
        c->pending.push_back(slot);
    }
}

bool float_dtype(int dt) { return dt == LT_F32 || dt == LT_BF16; }

bool valid_dtype(int dt) { return dt >= LT_F32 && dt <= LT_U32; }

lt_status check_shape(lt_ctx *c, int rank, const int64_t *shape) {
    if (rank < 0 || rank > LT_MAX_RANK) return fail(c, LT_ERR_INVALID_ARG, "rank must be between 0 and LT_MAX_RANK");
    if (rank > 0 && !shape) return fail(c, LT_ERR_INVALID_ARG, "shape is null");
    for (int i = 0; i < rank; ++i)
        if (shape[i] < 0) return fail(c, LT_ERR_INVALID_ARG, "negative dimension");
    return LT_OK;
}

// Collect the tensors a barrier must materialise (Section 4: all live tensors with
// outstanding computation), in creation order.
void gather_roots(lt_ctx *c, std::vector<uint32_t> &roots, bool consume) {
    roots.clear();
    for (uint32_t slot : c->pending) {
        TensorRec &t = c->tensors[slot];
        if (consume) t.queued = false;
        if (t.live && !is_leaf(c->nodes[t.node])) roots.push_back(slot);
    }
    std::sort(roots.begin(), roots.end(),
              [c](uint32_t a, uint32_t b) { return c->tensors[a].seq < c->tensors[b].seq; });
    roots.erase(std::unique(roots.begin(), roots.end()), roots.end());
    if (consume) {
        c->pending.clear();
    }
}

// The pending list has been turned into roots: forget it.
void consume_pending(lt_ctx *c) {
    for (uint32_t slot : c->pending) c->tensors[slot].queued = false;
    c->pending.clear();
}

void release_donors(lt_ctx *c, const std::vector<uint32_t> &roots) {
    for (uint32_t slot : roots) {
        TensorRec &t = c->tensors[slot];
        if (t.donor != NONE) {
            buffer_unref(c, t.donor);
            t.donor = NONE;
        }
    }
}

// Remembers, for lt_replay, which tensors the graph being flushed reads and writes.  Called after the
// launches, while the root tensors still name their IR and their lt_assign donors.
void record_replay(lt_ctx *c, Plan *cached, Plan *plan, const Canonical &cg, const std::vector<uint32_t> &roots) {
    ReplayRecord &r = c->replay;
    r.plan = cached;
    r.exec = plan;
    r.why_not.clear();
    r.dyn = cg.dyn;
    r.params.assign(cg.param_node.size(), ReplayRecord::ParamRef());
    r.dyn_scalar.assign(cg.dyn.size(), ReplayRecord::Ref());
    r.roots.clear();
    // arena node -> a live tensor naming it (leaves read as they are, run-time scalars)
    std::vector<uint32_t> &by_node = c->stack_scratch;  // reused as a map: node -> slot + 1
    by_node.assign(c->nodes.size(), 0);
    for (uint32_t slot = 0; slot < c->tensors.size(); ++slot)
        if (c->tensors[slot].live) by_node[c->tensors[slot].node] = slot + 1;
    // buffer -> the first root (in creation order) that named it before lt_assign
    std::vector<uint32_t> &by_donor = c->donor_scratch;
    by_donor.assign(c->buffers.size(), 0);
    for (size_t k = roots.size(); k-- > 0;)
        if (c->tensors[roots[k]].donor != NONE) by_donor[c->tensors[roots[k]].donor] = roots[k] + 1;
    auto ref_of = [c](uint32_t slot, ReplayRecord::Ref &ref) {
        ref.slot = slot;
        ref.gen = c->tensors[slot].gen;
    };
    for (size_t i = 0; i < cg.param_node.size(); ++i) {
        const Node &leaf = c->nodes[cg.param_node[i]];
        ReplayRecord::ParamRef &pr = r.params[i];
        pr.dtype = leaf.dtype;
        pr.rank = leaf.rank;
        memcpy(pr.dims, leaf.dims, sizeof(pr.dims));
        if (by_node[cg.param_node[i]]) {
            ref_of(by_node[cg.param_node[i]] - 1, pr);
            continue;
        }
        // an in-place update: the tensor that named this buffer before lt_assign
        if (leaf.buffer < by_donor.size() && by_donor[leaf.buffer]) ref_of(by_donor[leaf.buffer] - 1, pr);
        if (pr.slot == NONE && r.why_not.empty()) r.why_not = "an input of the flushed graph was not named by any tensor";
    }
    for (const CNode &cn : cg.nodes)
        if (cn.op == N_SCALAR && cn.dyn >= 0 && by_node[cn.arena]) ref_of(by_node[cn.arena] - 1, r.dyn_scalar[cn.dyn]);
    for (uint32_t slot : roots) {
        ReplayRecord::Root root;
        ref_of(slot, root);
        root.output = cg.nodes[c->nodes[c->tensors[slot].node].canon].output;
        r.roots.push_back(root);
    }
    r.in_place_ok.assign(plan->outputs.size(), 0);
    for (const ReplayRecord::Root &root : r.roots) {
        const int32_t p = plan->outputs[root.output].donated_param;
        if (p >= 0 && r.params[p].slot == root.slot) r.in_place_ok[root.output] = 1;
    }
    by_node.clear();
}

// Drains the stream; afterwards, if a kernel with bounded device-side waits has run since the last look, reads the
// device status word: a wait that gave up is reported (and the word cleared) here.
lt_status sync_and_check(lt_ctx *c) {
    cudaError_t e = cudaStreamSynchronize(c->stream);
    if (e != cudaSuccess) return fail(c, LT_ERR_CUDA, std::string("cudaStreamSynchronize: ") + cudaGetErrorString(e));
    if (c->status_pending) {
        c->status_pending = false;
        unsigned int word = 0;
        e = lt_device_status_read(&word, 1);
        if (e != cudaSuccess) return fail(c, LT_ERR_CUDA, std::string("reading the device status word: ") + cudaGetErrorString(e));
        if (word & 1u)
            return fail(c, LT_ERR_DEVICE_TIMEOUT, "a kernel gave up waiting for an asynchronous copy into shared memory; results of that flush are incomplete");
    }
    return LT_OK;
}

void put_text(const std::string &s, char *buf, size_t cap, size_t *need) {
    if (need) *need = s.size() + 1;
    if (buf && cap) {
        size_t n = std::min(cap - 1, s.size());
        memcpy(buf, s.data(), n);
        buf[n] = 0;
    }
}

std::string shape_text(int dtype, const int64_t *dims, int rank) {
    std::string s = dtype_name(dtype);
    s += "[";
    for (int i = 0; i < rank; ++i) {
        if (i) s += ",";
        s += std::to_string(dims[i]);
    }
    s += "]";
    return s;
}

}  // namespace

namespace lt {

size_t dtype_size(int dt) { return dt == LT_BF16 ? 2 : dt == LT_U8 ? 1 : 4; }

const char *dtype_name(int dt) {
    static const char *n[] = {"f32", "bf16", "u8", "i32", "u32"};
    return dt >= 0 && dt <= 4 ? n[dt] : "?";
}

const char *op_name(int op) {
    switch (op) {
    case LT_OP_ADD: return "add"; case LT_OP_SUB: return "sub"; case LT_OP_MUL: return "mul";
    case LT_OP_DIV: return "div"; case LT_OP_MAX: return "max"; case LT_OP_MIN: return "min";
    case LT_OP_AND: return "and"; case LT_OP_OR: return "or"; case LT_OP_XOR: return "xor";
    case LT_OP_GT: return "gt"; case LT_OP_GE: return "ge"; case LT_OP_LT: return "lt";
    case LT_OP_LE: return "le"; case LT_OP_EQ: return "eq"; case LT_OP_NE: return "ne";
    case LT_OP_WHERE: return "where";
    case LT_OP_NEG: return "neg"; case LT_OP_ABS: return "abs"; case LT_OP_RELU: return "relu";
    case LT_OP_EXP: return "exp"; case LT_OP_LOG: return "log"; case LT_OP_TANH: return "tanh";
    case LT_OP_SQRT: return "sqrt"; case LT_OP_RSQRT: return "rsqrt"; case LT_OP_RECIP: return "recip";
    case LT_OP_SQUARE: return "square"; case LT_OP_SIGMOID: return "sigmoid";
    case LT_OP_GELU_TANH: return "gelu_tanh"; case LT_OP_NOT: return "not";
    case LT_OP_CONVERT: return "convert"; case LT_OP_IOTA: return "iota";
    case LT_OP_PHILOX_BITS: return "philox_bits";
    case LT_OP_ROW_SUM: return "row_sum"; case LT_OP_ROW_MAX: return "row_max"; case LT_OP_ROW_MIN: return "row_min";
    case LT_OP_COL_SUM: return "col_sum"; case LT_OP_COL_MAX: return "col_max"; case LT_OP_COL_MIN: return "col_min";
    case LT_OP_ALL_SUM: return "all_sum"; case LT_OP_ALL_MAX: return "all_max"; case LT_OP_ALL_MIN: return "all_min";
    case LT_OP_RESHAPE: return "reshape"; case LT_OP_NARROW: return "narrow"; case LT_OP_PERMUTE: return "permute";
    case LT_OP_UPDATE_SLICE: return "update_slice";
    case N_DEVICE_DATA: return "device_data"; case N_SCALAR: return "constant";
    default: return "?";
    }
}

int64_t shape_numel(const int64_t *dims, int rank) {
    int64_t n = 1;
    for (int i = 0; i < rank; ++i) n *= dims[i];
    return n;
}

lt_status fail(lt_ctx *c, lt_status s, const std::string &msg) {
    if (c) c->error = msg;
    return s;
}

uint32_t node_new(lt_ctx *c) {
    uint32_t id;
    if (!c->free_nodes.empty()) {
        id = c->free_nodes.back();
        c->free_nodes.pop_back();
        c->nodes[id] = Node();
    } else {
        id = (uint32_t)c->nodes.size();
        c->nodes.emplace_back();
    }
    return id;
}

void node_ref(lt_ctx *c, uint32_t n) { c->nodes[n].refs++; }

void node_unref(lt_ctx *c, uint32_t n) {
    // iterative: long chains (an unrolled loop, Section 4.2) must not recurse deeply
    std::vector<uint32_t> &stack = c->stack_scratch;
    size_t base = stack.size();
    stack.push_back(n);
    while (stack.size() > base) {
        uint32_t id = stack.back();
        stack.pop_back();
        Node &nd = c->nodes[id];
        if (--nd.refs > 0) continue;
        for (int i = 0; i < nd.n_in; ++i) stack.push_back(nd.in[i]);
        if (nd.op == N_DEVICE_DATA && nd.buffer != NONE) buffer_unref(c, nd.buffer);
        nd.op = 0;
        nd.n_in = 0;
        c->free_nodes.push_back(id);
    }
}

uint32_t buffer_new(lt_ctx *c, void *ptr, size_t bytes, bool owned) {
    uint32_t id;
    if (!c->free_buffers.empty()) {
        id = c->free_buffers.back();
        c->free_buffers.pop_back();
    } else {
        id = (uint32_t)c->buffers.size();
        c->buffers.emplace_back();
    }
    Buffer &b = c->buffers[id];
    b.ptr = ptr;
    b.bytes = bytes;
    b.refs = 1;
    b.owned = owned;
    return id;
}

void buffer_unref(lt_ctx *c, uint32_t b) {
    Buffer &buf = c->buffers[b];
    if (--buf.refs > 0) return;
    if (buf.owned && buf.ptr) ctx_free(c, buf.ptr);
    buf.ptr = nullptr;
    c->free_buffers.push_back(b);
}

// Device memory of the context.  Blocks the library has released are kept in a per-size pool (up to
// `pool_bytes` in total) and handed out again before the allocator is asked: everything runs on one
// stream, so a block freed after the last kernel using it was enqueued can be reused by the next
// flush at once.  In steady state (same graph every step) a flush makes no allocator call at all.
static void *raw_alloc(lt_ctx *c, size_t bytes) {
    c->stats.allocator_calls++;
    DeviceScope on_device(c->has_alloc ? LT_DEVICE_NONE : c->device);
    if (c->has_alloc) return c->alloc.alloc(bytes, (void *)c->stream, c->alloc.user);
    if (c->device == LT_DEVICE_NONE) return malloc(bytes);
    void *p = nullptr;
    if (cudaMallocAsync(&p, bytes, c->stream) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    return p;
}

static void raw_free(lt_ctx *c, void *p) {
    c->stats.allocator_calls++;
    DeviceScope on_device(c->has_alloc ? LT_DEVICE_NONE : c->device);
    if (c->has_alloc) c->alloc.free(p, (void *)c->stream, c->alloc.user);
    else if (c->device == LT_DEVICE_NONE) free(p);
    else cudaFreeAsync(p, c->stream);
}

void pool_trim(lt_ctx *c, size_t keep_bytes) {
    for (auto it = c->pool.begin(); it != c->pool.end() && c->pool_held > keep_bytes;) {
        std::vector<void *> &v = it->second;
        while (!v.empty() && c->pool_held > keep_bytes) {
            c->block_size.erase(v.back());
            raw_free(c, v.back());
            v.pop_back();
            c->pool_held -= it->first;
        }
        it = v.empty() ? c->pool.erase(it) : std::next(it);
    }
}

void *ctx_alloc(lt_ctx *c, size_t bytes) {
    if (bytes == 0) bytes = 16;
    bytes = (bytes + 511u) & ~(size_t)511u;
    auto it = c->pool.find(bytes);
    if (it != c->pool.end() && !it->second.empty()) {
        void *p = it->second.back();
        it->second.pop_back();
        c->pool_held -= bytes;
        return p;
    }
    void *p = raw_alloc(c, bytes);
    if (!p && c->pool_held) {  // give the pooled blocks back and try once more
        pool_trim(c, 0);
        p = raw_alloc(c, bytes);
    }
    if (p) c->block_size[p] = bytes;
    return p;
}

void ctx_free(lt_ctx *c, void *p) {
    if (!p) return;
    auto it = c->block_size.find(p);
    if (it != c->block_size.end() && c->opt.pool_bytes > 0 && c->pool_held + it->second <= (size_t)c->opt.pool_bytes) {
        c->pool[it->second].push_back(p);
        c->pool_held += it->second;
        return;
    }
    if (it != c->block_size.end()) c->block_size.erase(it);
    raw_free(c, p);
}

}  // namespace lt

// ======================================================================= trace matching
//
// Section 7 of the paper names the cost of re-tracing an unchanged program every step as the first thing to remove.
// lt_replay removes it on request; this removes most of it without being asked.  While a trace is recorded as usual
// its calls are also logged, operands named relative to the trace (TraceScript).  When the barrier has flushed it,
// the log is kept with the plan that ran and with where that plan's parameters, run-time values and results come
// from in the log.  The next trace is then only compared with the log, call by call: a call that repeats the logged
// one returns a handle that has no IR node behind it.  If the barrier finds the whole log repeated, it binds the plan
// directly -- nothing is canonicalised, hashed or looked up.  The first call that differs (or any call that wants to
// look at a tensor's computation) makes the calls matched so far for real, on the same handles, and recording goes on
// as usual; the trace being built becomes the next log.
namespace {

constexpr uint32_t TRACE_RELEASED_AT_ONCE = 0xfffffffeu;  // in bind_slot, for a release event

inline bool peek_slot(const lt_ctx *c, lt_tensor h, uint32_t *slot) {
    if ((uint16_t)(h >> 48) != c->tag) return false;
    uint32_t s = (uint32_t)(h & 0xffffffffu);
    if (s == 0 || s > c->tensors.size()) return false;
    s -= 1;
    const TensorRec &t = c->tensors[s];
    if (!t.live || (t.gen & 0xffffu) != (uint32_t)((h >> 32) & 0xffffu)) return false;
    *slot = s;
    return true;
}

// A trace begins: after a barrier that flushed something, or when matching is given up.
void trace_begin(lt_ctx *c, uint8_t mode) {
    TraceState &T = c->trace;
    T.mode = c->opt.trace_match ? mode : (uint8_t)TM_OFF;
    T.epoch++;
    T.cursor = 0;
    T.n_imports = T.n_nodes = 0;
    T.force_slot = NONE;
    T.log.clear();
    T.log_valid = true;
    T.bind_import_slot.clear();
    T.bind_node.clear();
    T.deferred_release.clear();
    T.virtual_scalars.clear();
    if (T.mode == TM_MATCH) {
        // indexed by event and written before they are read: what the last trace left in them does not matter
        const size_t n = T.script.events.size();
        T.bind_slot.resize(n);
        T.bind_val.resize(n);
        T.bind_val2.resize(n);
    } else {
        T.bind_slot.clear();
        T.bind_val.clear();
        T.bind_val2.clear();
    }
}

inline void trace_unsupported(lt_ctx *c) { c->trace.log_valid = false; }

void trace_forget_plan(lt_ctx *c, const Plan *plan) {
    if (c->trace.script.plan == plan) {
        c->trace.script.clear();
        if (c->trace.mode == TM_MATCH) c->trace.mode = TM_LEARN;  // (only ever reached between traces or while learning)
    }
}

// ---- learning: the trace is recorded as usual and logged

// Id of tensor `slot` in the trace being logged.  A tensor from before the trace is described once, when it is
// first used: what it is, and which of the trace's input nodes it names (two tensors may name the same one).
uint32_t trace_learn_tid(lt_ctx *c, uint32_t slot) {
    TraceState &T = c->trace;
    TensorRec &t = c->tensors[slot];
    if (t.trace_epoch == T.epoch) return t.trace_id;
    Node &nd = c->nodes[t.node];
    TraceImport im;
    if (!(nd.op == N_DEVICE_DATA || nd.op == N_SCALAR) || t.view_base != NONE) T.log_valid = false;
    im.op = nd.op;
    im.dtype = nd.dtype;
    im.rank = nd.rank;
    im.flags = nd.flags;
    memcpy(im.dims, nd.dims, sizeof(im.dims));
    im.sval = (nd.op == N_SCALAR && !(nd.flags & NF_DYNAMIC)) ? nd.sval : 0.0;
    if (nd.trace_epoch == T.epoch) {
        if (nd.trace_ref & TID_IMPORT) im.node_ordinal = nd.trace_ref & ~TID_IMPORT;
        else T.log_valid = false;  // made in this trace yet named by a tensor that was not: not expressible
    } else {
        im.node_ordinal = T.n_nodes++;
        im.fresh_node = true;
        nd.trace_epoch = T.epoch;
        nd.trace_ref = TID_IMPORT | im.node_ordinal;
    }
    t.trace_id = TID_IMPORT | (uint32_t)T.log.imports.size();
    t.trace_epoch = T.epoch;
    T.log.imports.push_back(im);
    return t.trace_id;
}

inline bool trace_learning(const lt_ctx *c) { return c->trace.mode == TM_LEARN && c->trace.log_valid; }

// the tensor in `slot` is the result of the event about to be appended
void trace_log_result(lt_ctx *c, uint32_t slot) {
    TraceState &T = c->trace;
    const uint32_t idx = (uint32_t)T.log.events.size();
    TensorRec &t = c->tensors[slot];
    t.trace_id = idx;
    t.trace_epoch = T.epoch;
    Node &nd = c->nodes[t.node];
    nd.trace_ref = idx;
    nd.trace_epoch = T.epoch;
    TraceResult res;
    res.dtype = nd.dtype;
    res.rank = nd.rank;
    memcpy(res.dims, nd.dims, sizeof(res.dims));
    T.log.results.push_back(res);
}

void trace_log_op(lt_ctx *c, int opcode, const uint32_t *in_slots, int n_in, const int64_t *attrs, int n_attrs, uint32_t out_slot) {
    TraceState &T = c->trace;
    if (n_attrs > 64 || T.log.events.size() >= (1u << 18)) {  // (a longer trace is not worth a log of tens of megabytes)
        T.log_valid = false;
        return;
    }
    TraceEvent ev;
    ev.kind = TE_OP;
    ev.op = (uint16_t)opcode;
    ev.n_in = (uint8_t)n_in;
    ev.n_attrs = (uint8_t)n_attrs;
    for (int i = 0; i < n_in; ++i) ev.in[i] = trace_learn_tid(c, in_slots[i]);
    ev.attr_off = (uint32_t)T.log.attrs.size();
    T.log.attrs.insert(T.log.attrs.end(), attrs, attrs + n_attrs);
    trace_log_result(c, out_slot);
    T.log.events.push_back(ev);
}

void trace_log_scalar(lt_ctx *c, uint32_t out_slot) {
    TraceState &T = c->trace;
    const Node &nd = c->nodes[c->tensors[out_slot].node];
    TraceEvent ev;
    ev.kind = TE_SCALAR;
    ev.dtype = nd.dtype;
    ev.flags = nd.flags;
    ev.sval = (nd.flags & NF_DYNAMIC) ? 0.0 : nd.sval;
    trace_log_result(c, out_slot);
    T.log.events.push_back(ev);
}

void trace_log_leaf(lt_ctx *c, uint32_t out_slot) {
    TraceState &T = c->trace;
    const Node &nd = c->nodes[c->tensors[out_slot].node];
    TraceEvent ev;
    ev.kind = TE_LEAF;
    ev.dtype = nd.dtype;
    ev.rank = nd.rank;
    ev.n_attrs = nd.rank;
    ev.attr_off = (uint32_t)T.log.attrs.size();
    T.log.attrs.insert(T.log.attrs.end(), nd.dims, nd.dims + nd.rank);
    trace_log_result(c, out_slot);
    T.log.events.push_back(ev);
}

void trace_log_pair(lt_ctx *c, uint8_t kind, uint32_t a, uint32_t b) {
    TraceState &T = c->trace;
    TraceEvent ev;
    ev.kind = kind;
    ev.in[0] = trace_learn_tid(c, a);
    if (kind == TE_ASSIGN) ev.in[1] = trace_learn_tid(c, b);
    T.log.events.push_back(ev);
    T.log.results.emplace_back();
}

// The barrier has run `ran` for the logged trace: keep the log, with where the plan's inputs and results are in it.
// Called while the roots still name their IR and `cg` describes it.  Returns false if something cannot be expressed.
bool trace_seal(lt_ctx *c, Plan *plan, const Plan *ran, const Canonical &cg, const std::vector<uint32_t> &roots) {
    TraceState &T = c->trace;
    if (T.mode != TM_LEARN || !T.log_valid || !c->view_slots.empty() || T.log.events.empty()) return false;
    TraceScript &S = T.log;
    S.param_src.resize(cg.param_node.size());
    for (size_t p = 0; p < cg.param_node.size(); ++p) {
        const Node &nd = c->nodes[cg.param_node[p]];
        if (nd.trace_epoch != T.epoch) return false;  // an input the trace never touched (pending from earlier)
        S.param_src[p] = nd.trace_ref;
    }
    S.dyn_src.assign(cg.dyn.size(), TraceScript::DynSrc());
    for (const CNode &cn : cg.nodes) {
        if (cn.dyn < 0) continue;
        const Node &nd = c->nodes[cn.arena];
        if (nd.trace_epoch != T.epoch) return false;
        S.dyn_src[cn.dyn].ref = nd.trace_ref;
        if (cn.op == LT_OP_PHILOX_BITS) {
            S.dyn_src[cn.dyn + 1].ref = nd.trace_ref;
            S.dyn_src[cn.dyn + 1].which = 1;
        }
    }
    S.roots.clear();
    for (uint32_t slot : roots) {
        const TensorRec &t = c->tensors[slot];
        if (t.trace_epoch != T.epoch) return false;
        TraceScript::Root r;
        r.tid = t.trace_id;
        r.output = cg.nodes[c->nodes[t.node].canon].output;
        S.roots.push_back(r);
    }
    // what lt_replay would need after a flush that only matched this trace
    const ReplayRecord &R = c->replay;
    auto tid_of = [&](uint32_t slot) -> uint32_t {
        if (slot == NONE || c->tensors[slot].trace_epoch != T.epoch) return NONE;
        return c->tensors[slot].trace_id;
    };
    S.replay_why_not = R.why_not;
    S.replay_param.resize(R.params.size());
    for (size_t i = 0; i < R.params.size(); ++i) {
        S.replay_param[i] = tid_of(R.params[i].slot);
        if (S.replay_param[i] == NONE && S.replay_why_not.empty()) S.replay_why_not = "an input of the flushed graph was not named by a tensor of the trace";
    }
    S.replay_dyn_scalar.resize(R.dyn_scalar.size());
    for (size_t k = 0; k < R.dyn_scalar.size(); ++k) S.replay_dyn_scalar[k] = tid_of(R.dyn_scalar[k].slot);
    S.replay_in_place_ok = R.in_place_ok;
    S.n_nodes = T.n_nodes;
    S.plan = plan;
    (void)ran;
    T.script = std::move(T.log);
    T.log.clear();
    return true;
}

// ---- matching

// Does tensor `slot` have id `want` in the trace being followed?  A tensor from before the trace is checked
// against the description logged at the same point.
bool trace_match_tid(lt_ctx *c, uint32_t slot, uint32_t want) {
    TraceState &T = c->trace;
    TensorRec &t = c->tensors[slot];
    if (t.trace_epoch == T.epoch) return t.trace_id == want;
    if (want != (TID_IMPORT | T.n_imports) || T.n_imports >= T.script.imports.size() || t.view_base != NONE || t.node == NONE) return false;
    const TraceImport &im = T.script.imports[T.n_imports];
    Node &nd = c->nodes[t.node];
    if (nd.op != im.op || nd.dtype != im.dtype || nd.rank != im.rank || ((nd.flags ^ im.flags) & NF_DYNAMIC)) return false;
    for (int i = 0; i < nd.rank; ++i)
        if (nd.dims[i] != im.dims[i]) return false;
    if (nd.op == N_SCALAR && !(nd.flags & NF_DYNAMIC) && memcmp(&nd.sval, &im.sval, sizeof(double)) != 0) return false;
    if (nd.trace_epoch == T.epoch) {
        if (im.fresh_node || nd.trace_ref != (TID_IMPORT | im.node_ordinal)) return false;
    } else {
        if (!im.fresh_node || im.node_ordinal != T.n_nodes) return false;
        nd.trace_epoch = T.epoch;
        nd.trace_ref = TID_IMPORT | T.n_nodes;
        T.bind_node.push_back(t.node);
        T.n_nodes++;
    }
    t.trace_id = want;
    t.trace_epoch = T.epoch;
    T.bind_import_slot.push_back(slot);
    T.n_imports++;
    return true;
}

// the result of matched event `index`: a live handle with no node behind it
uint32_t trace_virtual_tensor(lt_ctx *c, uint32_t index) {
    uint32_t slot;
    if (!c->free_tensors.empty()) {
        slot = c->free_tensors.back();
        c->free_tensors.pop_back();
    } else {
        slot = (uint32_t)c->tensors.size();
        c->tensors.emplace_back();
    }
    TensorRec &t = c->tensors[slot];
    t.node = NONE;
    t.gen += 1;
    t.donor = NONE;
    t.seq = c->next_seq++;
    t.live = true;
    t.queued = false;
    t.view_base = NONE;
    t.view_op = 0;
    t.version = 0;
    t.base_seen = 0;
    t.trace_id = index;
    t.trace_epoch = c->trace.epoch;
    t.vflags = TV_VIRTUAL;
    c->trace.bind_slot[index] = slot;
    return slot;
}

bool trace_match_op(lt_ctx *c, int opcode, const lt_tensor *in, int n_in, const int64_t *attrs, int n_attrs, lt_tensor *out) {
    TraceState &T = c->trace;
    if (T.cursor >= T.script.events.size() || n_in < 0 || n_in > 3 || n_attrs < 0) return false;
    const TraceEvent &ev = T.script.events[T.cursor];
    if (ev.kind != TE_OP || ev.op != opcode || ev.n_in != n_in || ev.n_attrs != n_attrs || (n_in && !in) || (n_attrs && !attrs)) return false;
    for (int i = 0; i < n_in; ++i) {
        uint32_t slot;
        if (!peek_slot(c, in[i], &slot) || !trace_match_tid(c, slot, ev.in[i])) return false;
    }
    const int64_t *want = T.script.attrs.data() + ev.attr_off;
    int first = 0;
    if (opcode == LT_OP_PHILOX_BITS && n_attrs >= 2) {  // seed and offset are run-time values
        T.bind_val[T.cursor].i = attrs[0];
        T.bind_val2[T.cursor].i = attrs[1];
        first = 2;
    }
    for (int i = first; i < n_attrs; ++i)
        if (attrs[i] != want[i]) return false;
    const uint32_t slot = trace_virtual_tensor(c, T.cursor);
    T.cursor++;
    c->stats.nodes_recorded++;
    *out = make_handle(c, slot);
    return true;
}

bool trace_match_scalar(lt_ctx *c, double value, lt_dtype dtype, bool force_dynamic, lt_tensor *out) {
    TraceState &T = c->trace;
    if (T.cursor >= T.script.events.size()) return false;
    const TraceEvent &ev = T.script.events[T.cursor];
    uint64_t bits;
    memcpy(&bits, &value, 8);
    const bool dynamic = force_dynamic || !(bits == 0ull || value == 1.0);
    if (ev.kind != TE_SCALAR || ev.dtype != (uint8_t)dtype || ((ev.flags & NF_DYNAMIC) != 0) != dynamic) return false;
    if (!dynamic && memcmp(&ev.sval, &value, sizeof(double)) != 0) return false;
    T.bind_val[T.cursor].d = value;
    const uint32_t slot = trace_virtual_tensor(c, T.cursor);
    T.virtual_scalars.push_back(slot);
    T.cursor++;
    c->stats.nodes_recorded++;
    *out = make_handle(c, slot);
    return true;
}

bool trace_match_assign(lt_ctx *c, lt_tensor dst, lt_tensor src) {
    TraceState &T = c->trace;
    if (T.cursor >= T.script.events.size()) return false;
    const TraceEvent &ev = T.script.events[T.cursor];
    uint32_t ds, ss;
    if (ev.kind != TE_ASSIGN || !peek_slot(c, dst, &ds) || !peek_slot(c, src, &ss)) return false;
    if (!trace_match_tid(c, ds, ev.in[0]) || !trace_match_tid(c, ss, ev.in[1])) return false;
    TensorRec &d = c->tensors[ds];
    if (!(d.vflags & TV_VIRTUAL)) d.vflags |= TV_ASSIGNED;  // still names its old leaf; the barrier gives it the new value
    T.cursor++;
    return true;
}

bool trace_match_release(lt_ctx *c, lt_tensor h) {
    TraceState &T = c->trace;
    if (T.cursor >= T.script.events.size()) return false;
    const TraceEvent &ev = T.script.events[T.cursor];
    uint32_t slot;
    if (ev.kind != TE_RELEASE || !peek_slot(c, h, &slot)) return false;
    const bool untouched = c->tensors[slot].trace_epoch != T.epoch;
    if (!trace_match_tid(c, slot, ev.in[0])) return false;
    TensorRec &t = c->tensors[slot];
    if (untouched) {
        // a tensor from before the trace that the trace has not used: nothing recorded depends on it, it goes at once
        t.live = false;
        t.queued = false;
        if (t.donor != NONE) {
            buffer_unref(c, t.donor);
            t.donor = NONE;
        }
        c->nodes[t.node].tensor_refs--;
        node_unref(c, t.node);
        t.node = NONE;
        c->free_tensors.push_back(slot);
        T.bind_slot[T.cursor] = TRACE_RELEASED_AT_ONCE;
        T.cursor++;
        return true;
    }
    t.live = false;  // the handle is dead; the slot is kept until the barrier so that the calls can still be made for real
    t.vflags |= TV_RELEASED;
    T.deferred_release.push_back(slot);
    T.cursor++;
    return true;
}

bool trace_match_leaf(lt_ctx *c, lt_dtype dtype, int rank, const int64_t *shape) {
    TraceState &T = c->trace;
    if (T.cursor >= T.script.events.size()) return false;
    const TraceEvent &ev = T.script.events[T.cursor];
    if (ev.kind != TE_LEAF || ev.dtype != (uint8_t)dtype || ev.rank != rank || rank < 0 || (rank && !shape)) return false;
    const int64_t *want = T.script.attrs.data() + ev.attr_off;
    for (int i = 0; i < rank; ++i)
        if (shape[i] != want[i]) return false;
    return true;
}

void trace_bind_leaf(lt_ctx *c, uint32_t slot) {  // the (real) leaf just made is the result of the matched event
    TraceState &T = c->trace;
    TensorRec &t = c->tensors[slot];
    t.trace_id = T.cursor;
    t.trace_epoch = T.epoch;
    Node &nd = c->nodes[t.node];
    nd.trace_ref = T.cursor;
    nd.trace_epoch = T.epoch;
    T.bind_slot[T.cursor] = slot;
    T.cursor++;
}

}  // namespace

extern "C" {
static lt_status new_scalar(lt_ctx *c, double value, lt_dtype dtype, bool force_dynamic, lt_tensor *out);
}

namespace {

// Gives up matching: the calls matched so far are made for real, each on the handle it returned.
void trace_materialise(lt_ctx *c) {
    TraceState &T = c->trace;
    if (T.mode != TM_MATCH) return;
    const uint32_t n = T.cursor;
    std::vector<TraceEvent> events(T.script.events.begin(), T.script.events.begin() + n);
    std::vector<int64_t> attrs;
    attrs.swap(T.script.attrs);
    std::vector<uint32_t> bslot, bimp, deferred;
    std::vector<DynValue> bval, bval2;
    bslot.swap(T.bind_slot);
    bimp.swap(T.bind_import_slot);
    bval.swap(T.bind_val);
    bval2.swap(T.bind_val2);
    deferred.swap(T.deferred_release);
    std::vector<TraceImport> old_imports;
    old_imports.swap(T.script.imports);
    T.script.clear();
    if (n) {
        c->stats.traces_diverged++;
        if (++T.streak >= 4) T.streak = 0, T.backoff = 16;
    }
    trace_begin(c, TM_LEARN);
    if (!n) return;
    for (uint32_t slot : deferred) c->tensors[slot].live = true;  // released again below, for real
    for (uint32_t slot : bimp) c->tensors[slot].vflags = 0;
    uint64_t counted = 0;
    auto slot_of = [&](uint32_t tid) { return (tid & TID_IMPORT) ? bimp[tid & ~TID_IMPORT] : bslot[tid]; };
    lt_status st = LT_OK;
    for (uint32_t e = 0; e < n && st == LT_OK; ++e) {
        const TraceEvent &ev = events[e];
        lt_tensor out = 0;
        if (ev.kind == TE_OP) {
            lt_tensor in[3] = {0, 0, 0};
            for (int i = 0; i < ev.n_in; ++i) in[i] = make_handle(c, slot_of(ev.in[i]));
            int64_t a[64];
            for (int i = 0; i < ev.n_attrs; ++i) a[i] = attrs[ev.attr_off + i];
            if (ev.op == LT_OP_PHILOX_BITS && ev.n_attrs >= 2) a[0] = bval[e].i, a[1] = bval2[e].i;
            T.force_slot = bslot[e];
            st = lt_op(c, ev.op, in, ev.n_in, a, ev.n_attrs, &out);
            ++counted;
        } else if (ev.kind == TE_SCALAR) {
            T.force_slot = bslot[e];
            st = new_scalar(c, bval[e].d, (lt_dtype)ev.dtype, (ev.flags & NF_DYNAMIC) != 0, &out);
            ++counted;
        } else if (ev.kind == TE_ASSIGN) {
            st = lt_assign(c, make_handle(c, slot_of(ev.in[0])), make_handle(c, slot_of(ev.in[1])));
        } else if (ev.kind == TE_RELEASE) {
            if (bslot[e] == TRACE_RELEASED_AT_ONCE) {
                // the tensor is gone already; what the log says about it is what the followed log said
                if (trace_learning(c)) {
                    TraceImport im = old_imports[ev.in[0] & ~TID_IMPORT];
                    if (im.fresh_node) im.node_ordinal = T.n_nodes++;
                    TraceEvent copy = ev;
                    copy.in[0] = TID_IMPORT | (uint32_t)T.log.imports.size();
                    T.log.imports.push_back(im);
                    T.log.events.push_back(copy);
                    T.log.results.emplace_back();
                    T.bind_slot.push_back(NONE);
                    T.bind_import_slot.push_back(NONE);
                }
            } else {
                st = lt_release(c, make_handle(c, slot_of(ev.in[0])));
            }
        } else {  // the leaf exists; it only has to be in the new log
            if (trace_learning(c)) {
                trace_log_leaf(c, bslot[e]);
                T.bind_slot.push_back(bslot[e]);
            }
        }
        T.force_slot = NONE;
    }
    c->stats.nodes_recorded -= counted;  // they were counted when they were matched
    if (st != LT_OK) {
        // cannot happen for calls that were accepted once; if it does, say so and stop matching for good
        fprintf(stderr, "[lazytensor] internal error: a matched trace could not be rebuilt (%s)\n", c->error.c_str());
        c->opt.trace_match = 0;
        T.mode = TM_OFF;
    }
}

inline void trace_materialise_if_started(lt_ctx *c) {
    if (c->trace.mode == TM_MATCH && c->trace.cursor) trace_materialise(c);
}

// The barrier of a trace that repeated the logged one to the end: binds and runs the logged plan.
// False: something differs after all (the caller rebuilds the trace and takes the usual path).
bool trace_barrier(lt_ctx *c, int blocking, lt_status *result) {
    TraceState &T = c->trace;
    TraceScript &S = T.script;
    if (T.cursor != S.events.size() || !S.plan || T.n_imports != S.imports.size() || T.n_nodes != S.n_nodes) return false;
    Plan *plan = S.plan;
    Canonical &cg = c->canon;
    auto slot_of = [&](uint32_t tid) { return (tid & TID_IMPORT) ? T.bind_import_slot[tid & ~TID_IMPORT] : T.bind_slot[tid]; };
    cg.param_node.resize(S.param_src.size());
    for (size_t p = 0; p < S.param_src.size(); ++p) {
        const uint32_t ref = S.param_src[p];
        cg.param_node[p] = (ref & TID_IMPORT) ? T.bind_node[ref & ~TID_IMPORT] : c->tensors[T.bind_slot[ref]].node;
    }
    // the roots are taken in creation order: the tensors from before the trace must still be in the logged order
    uint64_t last_seq = 0;
    for (const TraceScript::Root &r : S.roots) {
        const TensorRec &t = c->tensors[slot_of(r.tid)];
        if (!t.live || t.seq <= last_seq) return false;
        last_seq = t.seq;
    }
    Plan *ran = plan;
    if (!long_rows_runnable(c, *plan, cg)) {
        if (!plan->split) return false;
        ran = plan->split.get();
    }
    // a result written in place: the tensor that receives it must be the only one naming the buffer (Section 4.3)
    std::vector<uint8_t> &receiver = c->param_taken;  // per output: a root that names the donated input and was assigned to
    receiver.assign(plan->outputs.size(), 0);
    for (const TraceScript::Root &r : S.roots) {
        const int32_t p = plan->outputs[r.output].donated_param;
        if (p < 0) continue;
        const TensorRec &t = c->tensors[slot_of(r.tid)];
        if (!(t.vflags & TV_VIRTUAL) && (t.vflags & TV_ASSIGNED) && t.node == cg.param_node[p]) receiver[r.output] = 1;
    }
    for (size_t k = 0; k < plan->outputs.size(); ++k) {
        const int32_t p = plan->outputs[k].donated_param;
        if (p < 0) continue;
        const Node &leaf = c->nodes[cg.param_node[p]];
        if (!receiver[k] || leaf.tensor_refs != 1 || c->buffers[leaf.buffer].refs != 1) return false;
    }
    cg.dyn.resize(S.dyn_src.size());
    for (size_t k = 0; k < S.dyn_src.size(); ++k) {
        const TraceScript::DynSrc &d = S.dyn_src[k];
        if (d.ref & TID_IMPORT) cg.dyn[k].d = c->nodes[T.bind_node[d.ref & ~TID_IMPORT]].sval;
        else cg.dyn[k] = d.which ? T.bind_val2[d.ref] : T.bind_val[d.ref];
    }
    {
        Timer tm(c->stats.ns_bind_launch);
        lt_status s = execute_plan(c, *ran, cg, nullptr);
        if (s) {
            *result = s;  // nothing was rebound: the barrier can be called again
            return true;
        }
    }
    c->stats.barriers++;
    c->stats.cache_hits++;
    c->stats.traces_matched++;
    T.streak = 0;
    plan->last_used = ++c->use_clock;
    c->last_plan = plan;
    if (c->opt.log >= 2)
        fprintf(stderr, "[lazytensor] barrier %llu: trace matched (%zu calls), %zu launches\n", (unsigned long long)c->stats.barriers,
                S.events.size(), ran->launches.size());
    {
        Timer tm(c->stats.ns_rebind);
        // what lt_replay needs, while the input leaves are still there
        ReplayRecord &R = c->replay;
        auto ref_of = [&](uint32_t tid, ReplayRecord::Ref &ref) {
            ref.slot = NONE;
            ref.gen = 0;
            if (tid == NONE) return;
            ref.slot = slot_of(tid);
            ref.gen = c->tensors[ref.slot].gen;
        };
        R.plan = plan;
        R.exec = ran;
        R.why_not = S.replay_why_not;
        R.dyn = cg.dyn;
        R.params.assign(S.replay_param.size(), ReplayRecord::ParamRef());
        for (size_t i = 0; i < S.replay_param.size(); ++i) {
            const Node &leaf = c->nodes[cg.param_node[i]];
            R.params[i].dtype = leaf.dtype;
            R.params[i].rank = leaf.rank;
            memcpy(R.params[i].dims, leaf.dims, sizeof(leaf.dims));
            ref_of(S.replay_param[i], R.params[i]);
        }
        R.dyn_scalar.assign(S.replay_dyn_scalar.size(), ReplayRecord::Ref());
        for (size_t k = 0; k < S.replay_dyn_scalar.size(); ++k) ref_of(S.replay_dyn_scalar[k], R.dyn_scalar[k]);
        R.roots.clear();
        for (const TraceScript::Root &r : S.roots) {
            ReplayRecord::Root root;
            ref_of(r.tid, root);
            root.output = r.output;
            R.roots.push_back(root);
        }
        R.in_place_ok = S.replay_in_place_ok;
        // results: new leaves, as after any flush
        const size_t n_out = ran->outputs.size();
        // A result written in place whose only root is the tensor that names the buffer (checked above: alone) already
        // lives where that tensor's leaf points: the leaf stays, nothing is rebound.
        std::vector<uint32_t> &sharers = c->stack_scratch;  // per output: how many roots receive it
        sharers.assign(n_out, 0);
        for (const TraceScript::Root &r : S.roots) sharers[r.output]++;
        std::vector<uint32_t> new_nodes(n_out, NONE);
        for (size_t k = 0; k < n_out; ++k) {
            const OutputPlan &op = ran->outputs[k];
            if (op.donated_param >= 0 && sharers[k] == 1) continue;
            const uint32_t n = node_new(c);
            Node &nd = c->nodes[n];
            nd.op = N_DEVICE_DATA;
            nd.dtype = op.dtype;
            nd.rank = op.rank;
            memcpy(nd.dims, op.dims, sizeof(nd.dims));
            if (op.donated_param >= 0) {
                const uint32_t b = c->nodes[cg.param_node[op.donated_param]].buffer;
                c->buffers[b].refs++;
                nd.buffer = b;
            } else {
                nd.buffer = buffer_new(c, c->out_ptr[k], op.bytes, true);
            }
            nd.refs = 1;
            new_nodes[k] = n;
        }
        for (const TraceScript::Root &r : S.roots) {
            TensorRec &t = c->tensors[slot_of(r.tid)];
            const uint32_t nn = new_nodes[r.output];
            if (nn == NONE) {
                t.vflags = 0;
                t.version++;
                continue;
            }
            const uint32_t old = (t.vflags & TV_VIRTUAL) ? NONE : t.node;
            t.node = nn;
            t.vflags = 0;
            node_ref(c, nn);
            c->nodes[nn].tensor_refs++;
            if (old != NONE) {
                t.version++;
                c->nodes[old].tensor_refs--;
                node_unref(c, old);
            }
        }
        // scalars made during the trace and still alive become real constants
        for (uint32_t slot : T.virtual_scalars) {
            TensorRec &t = c->tensors[slot];
            if (!t.live || !(t.vflags & TV_VIRTUAL) || t.trace_epoch != T.epoch) continue;
            const TraceEvent &ev = S.events[t.trace_id];
            const uint32_t n = node_new(c);
            Node &nd = c->nodes[n];
            nd.op = N_SCALAR;
            nd.dtype = ev.dtype;
            nd.rank = 0;
            nd.flags = ev.flags;
            nd.sval = T.bind_val[t.trace_id].d;
            nd.refs = 1;
            nd.tensor_refs = 1;
            t.node = n;
            t.vflags = 0;
        }
        // the releases of the trace
        for (uint32_t slot : T.deferred_release) {
            TensorRec &t = c->tensors[slot];
            if (!(t.vflags & TV_VIRTUAL)) {  // a tensor from before the trace that the trace also read: its node goes now, like the rest of the flushed IR
                if (t.donor != NONE) {
                    buffer_unref(c, t.donor);
                    t.donor = NONE;
                }
                c->nodes[t.node].tensor_refs--;
                node_unref(c, t.node);
            }
            t.vflags = 0;
            t.node = NONE;
            t.queued = false;
            c->free_tensors.push_back(slot);
        }
        for (uint32_t slot : T.bind_import_slot) c->tensors[slot].vflags = 0;
        for (uint32_t n : new_nodes)
            if (n != NONE) node_unref(c, n);
        sharers.clear();
    }
    trace_begin(c, TM_MATCH);
    *result = (blocking && c->device != LT_DEVICE_NONE) ? sync_and_check(c) : LT_OK;
    return true;
}

}  // namespace

// ======================================================================= C ABI

extern "C" {

const char *lt_version(void) { return "lazytensor-b200 0.1"; }

const char *lt_last_error(lt_ctx *ctx) { return ctx ? ctx->error.c_str() : "null context"; }

lt_status lt_ctx_create(int device, void *cuda_stream, const lt_allocator *allocator, lt_ctx **out) {
    if (!out) return LT_ERR_INVALID_ARG;
    *out = nullptr;
    if (device < LT_DEVICE_NONE) return LT_ERR_INVALID_ARG;
    lt_ctx *c = new (std::nothrow) lt_ctx();
    if (!c) return LT_ERR_OOM;
    c->device = device;
    c->stream = (cudaStream_t)cuda_stream;
    c->tag = (uint16_t)(g_next_tag.fetch_add(1) & 0xffffu);
    if (c->tag == 0) c->tag = (uint16_t)(g_next_tag.fetch_add(1) & 0xffffu);
    if (allocator) {
        if (!allocator->alloc || !allocator->free) {
            delete c;
            return LT_ERR_INVALID_ARG;
        }
        c->alloc = *allocator;
        c->has_alloc = true;
    }
    auto env_opt = [](const char *name, int64_t *dst) {
        const char *v = getenv(name);
        if (v && *v) *dst = strtoll(v, nullptr, 10);
    };
    env_opt("LT_FUSION", &c->opt.fusion);
    env_opt("LT_VERIFY", &c->opt.verify);
    env_opt("LT_FAST_MATH", &c->opt.fast_math);
    env_opt("LT_HORIZONTAL", &c->opt.horizontal);
    env_opt("LT_LOG", &c->opt.log);
    if (device != LT_DEVICE_NONE) {
        DeviceScope on_device(device);  // the caller's current device is put back when the call returns
        cudaError_t e = on_device.ok() ? cudaSuccess : cudaErrorInvalidDevice;
        int sms = 0;
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
        if (e == cudaSuccess) e = lt_kernel_setup(LT_MAX_STAGE_BYTES);
        if (e == cudaSuccess) e = lt_kernel_occupancy(&c->occ_ew, &c->occ_row, &c->occ_multi);
        if (e != cudaSuccess) {
            // no usable device: report instead of falling back to anything
            fprintf(stderr, "lt_ctx_create: CUDA device %d unusable: %s\n", device, cudaGetErrorString(e));
            cudaGetLastError();
            delete c;
            return LT_ERR_CUDA;
        }
        c->sm_count = sms;
        if (c->occ_ew < 1) c->occ_ew = 1;
        if (c->occ_row < 1) c->occ_row = 1;
        if (c->occ_multi < 1) c->occ_multi = 1;
    }
    *out = c;
    return LT_OK;
}

lt_status lt_ctx_destroy(lt_ctx *c) {
    if (!c) return LT_ERR_INVALID_ARG;
    DeviceScope on_device(c->device);
    if (c->device != LT_DEVICE_NONE) cudaStreamSynchronize(c->stream);
    for (auto &t : c->timed) {
        cudaEventDestroy(t.start);
        cudaEventDestroy(t.stop);
    }
    for (auto e : c->event_pool) cudaEventDestroy(e);
    for (auto &b : c->buffers)
        if (b.owned && b.ptr && b.refs > 0) ctx_free(c, b.ptr);
    pool_trim(c, 0);
    delete c;
    return LT_OK;
}

lt_status lt_ctx_set_option(lt_ctx *c, const char *key, int64_t value) {
    if (!c || !key) return LT_ERR_INVALID_ARG;
    // a logged trace is tied to the plan made under the options of its time
    trace_materialise(c);
    c->trace.script.clear();
    if (c->trace.mode == TM_MATCH) c->trace.mode = TM_LEARN;
    if (!strcmp(key, "trace_match")) {
        c->opt.trace_match = value;
        c->trace.mode = value ? (uint8_t)TM_LEARN : (uint8_t)TM_OFF;
        c->trace.log_valid = false;  // (a trace may be half recorded: start logging with the next one)
        return LT_OK;
    }
    if (!strcmp(key, "fusion")) c->opt.fusion = value;
    else if (!strcmp(key, "verify")) c->opt.verify = value;
    else if (!strcmp(key, "fast_math")) c->opt.fast_math = value;
    else if (!strcmp(key, "horizontal")) c->opt.horizontal = value;
    else if (!strcmp(key, "cache_capacity")) c->opt.cache_capacity = value;
    else if (!strcmp(key, "ieee")) c->opt.ieee = value;
    else if (!strcmp(key, "debug.waves")) c->opt.waves = value;
    else if (!strcmp(key, "debug.stage")) c->opt.stage = value;
    else if (!strcmp(key, "log")) c->opt.log = value;
    else if (!strcmp(key, "pool_bytes")) {
        c->opt.pool_bytes = value;
        pool_trim(c, value > 0 ? (size_t)value : 0);
    }
    else if (!strcmp(key, "compiled")) c->opt.compiled = value;
    else if (!strcmp(key, "debug.compiled_u")) c->opt.compiled_u = value;
    else if (!strcmp(key, "debug.compiled_row_u")) c->opt.compiled_row_u = value;
    else if (!strcmp(key, "debug.compiled_depth")) c->opt.compiled_depth = value;
    else if (!strcmp(key, "debug.long_l2_ahead")) c->opt.long_l2_ahead = value;
    else if (!strcmp(key, "debug.ignore_table")) c->opt.ignore_table = value;
    else if (!strcmp(key, "debug.cluster")) c->opt.cluster = value;
    else if (!strcmp(key, "debug.cluster_vectors")) c->opt.cluster_vectors = value;
    else if (!strcmp(key, "specialise")) c->opt.specialise = value;
    else if (!strcmp(key, "specialise_after")) c->opt.specialise_after = value;
    else if (!strcmp(key, "wait_limit_ms")) c->wait_limit_ns = value > 0 ? value * 1000000ll : 1;
    else return fail(c, LT_ERR_INVALID_ARG, std::string("unknown option ") + key);
    return LT_OK;
}

static lt_status new_device_tensor(lt_ctx *c, void *dptr, bool owned, lt_dtype dtype, int rank, const int64_t *shape,
                                   lt_tensor *out) {
    size_t bytes = (size_t)shape_numel(shape, rank) * dtype_size(dtype);
    uint32_t n = node_new(c);
    Node &nd = c->nodes[n];
    nd.op = N_DEVICE_DATA;
    nd.dtype = (uint8_t)dtype;
    nd.rank = (uint8_t)rank;
    for (int i = 0; i < rank; ++i) nd.dims[i] = shape[i];
    nd.buffer = buffer_new(c, dptr, bytes, owned);
    uint32_t slot = tensor_new(c, n);
    *out = make_handle(c, slot);
    return LT_OK;
}

lt_status lt_tensor_from_device(lt_ctx *c, void *dptr, lt_dtype dtype, int rank, const int64_t *shape,
                                lt_tensor *out) {
    if (!c || !out) return LT_ERR_INVALID_ARG;
    RecordTimer tm(c);
    if (!valid_dtype(dtype)) return fail(c, LT_ERR_DTYPE, "unknown dtype");
    lt_status s = check_shape(c, rank, shape);
    if (s) return s;
    if (!dptr && shape_numel(shape, rank) > 0) return fail(c, LT_ERR_INVALID_ARG, "device pointer is null");
    c->stats.nodes_recorded++;
    bool matched = false;
    if (c->trace.mode == TM_MATCH) {
        matched = trace_match_leaf(c, dtype, rank, shape);
        if (!matched) trace_materialise(c);
    }
    s = new_device_tensor(c, dptr, false, dtype, rank, shape, out);
    if (s) return s;
    const uint32_t slot = (uint32_t)(*out & 0xffffffffu) - 1;
    if (matched) trace_bind_leaf(c, slot);
    else if (trace_learning(c)) {
        trace_log_leaf(c, slot);
        c->trace.bind_slot.push_back(slot);
    }
    return LT_OK;
}

lt_status lt_tensor_from_host(lt_ctx *c, const void *hptr, lt_dtype dtype, int rank, const int64_t *shape,
                              lt_tensor *out) {
    if (!c || !out) return LT_ERR_INVALID_ARG;
    if (!valid_dtype(dtype)) return fail(c, LT_ERR_DTYPE, "unknown dtype");
    lt_status s = check_shape(c, rank, shape);
    if (s) return s;
    if (c->device == LT_DEVICE_NONE) return fail(c, LT_ERR_UNSUPPORTED, "context has no device");
    trace_materialise(c);
    trace_unsupported(c);
    DeviceScope on_device(c->device);
    if (!on_device.ok()) return fail(c, LT_ERR_CUDA, "cudaSetDevice failed for the context's device");
    size_t bytes = (size_t)shape_numel(shape, rank) * dtype_size(dtype);
    if (!hptr && bytes) return fail(c, LT_ERR_INVALID_ARG, "host pointer is null");
    void *d = ctx_alloc(c, bytes);
    if (!d) return fail(c, LT_ERR_OOM, "allocator returned null");
    if (bytes) {
        cudaError_t e = cudaMemcpyAsync(d, hptr, bytes, cudaMemcpyHostToDevice, c->stream);
        if (e != cudaSuccess) {
            ctx_free(c, d);
            return fail(c, LT_ERR_CUDA, std::string("cudaMemcpyAsync: ") + cudaGetErrorString(e));
        }
    }
    c->stats.nodes_recorded++;
    return new_device_tensor(c, d, true, dtype, rank, shape, out);
}

static lt_status new_scalar(lt_ctx *c, double value, lt_dtype dtype, bool force_dynamic, lt_tensor *out) {
    if (!c || !out) return LT_ERR_INVALID_ARG;
    RecordTimer tm(c);
    if (!valid_dtype(dtype)) return fail(c, LT_ERR_DTYPE, "unknown dtype");
    if (c->trace.mode == TM_MATCH) {
        if (trace_match_scalar(c, value, dtype, force_dynamic, out)) return LT_OK;
        trace_materialise(c);
    }
    uint32_t n = node_new(c);
    Node &nd = c->nodes[n];
    nd.op = N_SCALAR;
    nd.dtype = (uint8_t)dtype;
    nd.rank = 0;
    nd.sval = value;
    // Section 4.1 heuristic: only 0 and 1 are baked into the graph
    uint64_t bits;
    memcpy(&bits, &value, 8);
    bool special = bits == 0ull || value == 1.0;
    if (force_dynamic || !special) nd.flags |= NF_DYNAMIC;
    c->stats.nodes_recorded++;
    uint32_t slot = tensor_new(c, n);
    if (trace_learning(c)) {
        trace_log_scalar(c, slot);
        c->trace.bind_slot.push_back(slot);
    }
    *out = make_handle(c, slot);
    return LT_OK;
}

lt_status lt_scalar(lt_ctx *c, double value, lt_dtype dtype, lt_tensor *out) {
    return new_scalar(c, value, dtype, false, out);
}

lt_status lt_scalar_dynamic(lt_ctx *c, double value, lt_dtype dtype, lt_tensor *out) {
    return new_scalar(c, value, dtype, true, out);
}

// class of operand shape relative to the result shape: 0 same, 1 scalar, 2 column vector, 3 row scalar, -1 none
static int operand_class(const Node &a, const int64_t *od, int orank) {
    int64_t na = shape_numel(a.dims, a.rank);
    bool same = a.rank == orank;
    for (int i = 0; same && i < orank; ++i) same = a.dims[i] == od[i];
    if (same) return 0;
    if (na == 1) return 1;
    if (orank >= 1 && a.rank >= 1 && a.rank <= orank && a.dims[a.rank - 1] == od[orank - 1]) {
        bool ones = true;
        for (int i = 0; i + 1 < a.rank; ++i) ones = ones && a.dims[i] == 1;
        if (ones) return 2;
    }
    if (a.rank == orank && orank >= 1 && a.dims[orank - 1] == 1) {
        bool lead = true;
        for (int i = 0; i + 1 < orank; ++i) lead = lead && a.dims[i] == od[i];
        if (lead) return 3;
    }
    return -1;
}

// result shape of broadcasting the operands against each other (dimensions aligned at the right)
static bool broadcast_shape(const Node *const *ops, int n, int64_t *od, int *orank) {
    int r = 0;
    for (int k = 0; k < n; ++k) r = std::max(r, (int)ops[k]->rank);
    for (int i = 0; i < r; ++i) od[i] = 1;
    for (int k = 0; k < n; ++k) {
        const Node &a = *ops[k];
        for (int i = 0; i < a.rank; ++i) {
            int o = r - a.rank + i;
            if (a.dims[i] == 1) continue;
            if (od[o] == 1) od[o] = a.dims[i];
            else if (od[o] != a.dims[i]) return false;
        }
    }
    *orank = r;
    return true;
}

static bool scalar_fits(const Node &s, int dtype) {
    if (s.op != N_SCALAR) return true;
    if (float_dtype(dtype)) return true;
    double v = s.sval;
    if (v != std::floor(v)) return false;
    if (dtype == LT_U8) return v >= 0 && v <= 255;
    if (dtype == LT_I32) return v >= -2147483648.0 && v <= 2147483647.0;
    return v >= 0 && v <= 4294967295.0;
}


// ---- shape operations (pure IR nodes) and views (Section 4.4)

static uint64_t pack_perm(const int *perm, int rank) {
    uint64_t v = 0;
    for (int i = 0; i < rank; ++i) v |= (uint64_t)(perm[i] & 0xf) << (4 * i);
    return v;
}

// Appends the node `opcode`(src [, upd]) with the given attributes; shapes are validated here.  For RESHAPE of
// materialised data no operation is recorded: the result is another leaf over the same buffer.
static lt_status record_shape_op(lt_ctx *c, int opcode, uint32_t src, uint32_t upd, int64_t a0, int64_t a1, int rank,
                                 const int64_t *dims, uint32_t *out_node) {
    const Node s = c->nodes[src];  // copy: the arena may grow below
    if (s.op == N_SCALAR) return fail(c, LT_ERR_INVALID_ARG, "shape operations need a tensor, not a constant");
    int64_t od[LT_MAX_RANK] = {0};
    int orank = s.rank;
    if (opcode == LT_OP_RESHAPE) {
        lt_status st = check_shape(c, rank, dims);
        if (st) return st;
        if (shape_numel(dims, rank) != shape_numel(s.dims, s.rank)) return fail(c, LT_ERR_SHAPE, "reshape must keep the number of elements");
        orank = rank;
        for (int i = 0; i < rank; ++i) od[i] = dims[i];
        if (s.op == N_DEVICE_DATA) {
            uint32_t n = node_new(c);
            Node &nd = c->nodes[n];
            nd.op = N_DEVICE_DATA;
            nd.dtype = s.dtype;
            nd.rank = (uint8_t)orank;
            for (int i = 0; i < orank; ++i) nd.dims[i] = od[i];
            nd.buffer = s.buffer;
            c->buffers[s.buffer].refs++;
            *out_node = n;
            return LT_OK;
        }
    } else if (opcode == LT_OP_NARROW) {
        const int64_t dim = a0, start = a1, len = rank;  // (length travels in `rank`)
        if (dim < 0 || dim >= s.rank) return fail(c, LT_ERR_INVALID_ARG, "narrow: dimension out of range");
        if (start < 0 || len < 1 || start + len > s.dims[dim]) return fail(c, LT_ERR_SHAPE, "narrow: slice outside the dimension");
        memcpy(od, s.dims, sizeof(od));
        od[dim] = len;
    } else if (opcode == LT_OP_PERMUTE) {
        bool seen[LT_MAX_RANK] = {false};
        for (int i = 0; i < s.rank; ++i) {
            const int p = (int)((a0 >> (4 * i)) & 0xf);
            if (p >= s.rank || seen[p]) return fail(c, LT_ERR_INVALID_ARG, "permute: not a permutation of the dimensions");
            seen[p] = true;
            od[i] = s.dims[p];
        }
    } else {  // UPDATE_SLICE
        const Node &u = c->nodes[upd];
        const int64_t dim = a0, start = a1;
        if (u.op == N_SCALAR || u.dtype != s.dtype || u.rank != s.rank) return fail(c, LT_ERR_SHAPE, "update_slice: update must match the base's dtype and rank");
        if (dim < 0 || dim >= s.rank) return fail(c, LT_ERR_INVALID_ARG, "update_slice: dimension out of range");
        for (int i = 0; i < s.rank; ++i)
            if (i != dim && u.dims[i] != s.dims[i]) return fail(c, LT_ERR_SHAPE, "update_slice: update must match the base outside the sliced dimension");
        if (start < 0 || start + u.dims[dim] > s.dims[dim]) return fail(c, LT_ERR_SHAPE, "update_slice: slice outside the dimension");
        memcpy(od, s.dims, sizeof(od));
    }
    uint32_t n = node_new(c);
    Node &nd = c->nodes[n];
    nd.op = (uint16_t)opcode;
    nd.dtype = s.dtype;
    nd.rank = (uint8_t)orank;
    for (int i = 0; i < orank; ++i) nd.dims[i] = od[i];
    nd.attr[0] = a0;
    nd.attr[1] = a1;
    nd.n_in = opcode == LT_OP_UPDATE_SLICE ? 2 : 1;
    nd.in[0] = src;
    node_ref(c, src);
    if (opcode == LT_OP_UPDATE_SLICE) {
        nd.in[1] = upd;
        node_ref(c, upd);
    }
    c->stats.nodes_recorded++;
    *out_node = n;
    return LT_OK;
}

// `slot` from now on denotes the computation `node` (the core of lt_assign).
static void repoint_tensor(lt_ctx *c, uint32_t slot, uint32_t node, bool keep_donor) {
    TensorRec &d = c->tensors[slot];
    if (d.node == node) return;
    const Node &dn = c->nodes[d.node];
    if (keep_donor && dn.op == N_DEVICE_DATA && dn.buffer != NONE) {
        if (d.donor != NONE) buffer_unref(c, d.donor);
        d.donor = dn.buffer;
        c->buffers[d.donor].refs++;
    }
    const uint32_t old = d.node;
    d.node = node;
    node_ref(c, node);
    c->nodes[node].tensor_refs++;
    c->nodes[old].tensor_refs--;
    node_unref(c, old);
    queue_pending(c, slot);
}

static bool view_base_alive(const lt_ctx *c, const TensorRec &t) {
    return t.view_base != NONE && t.view_base < c->tensors.size() && c->tensors[t.view_base].live &&
           c->tensors[t.view_base].gen == t.view_base_gen;
}

// the view operation of tensor `t` applied to `src`
static lt_status apply_view_op(lt_ctx *c, const TensorRec &t, uint32_t src, uint32_t *out_node) {
    const Node &cur = c->nodes[t.node];  // the view's shape does not change
    if (t.view_op == LT_OP_RESHAPE) {
        int64_t dims[LT_MAX_RANK];
        memcpy(dims, cur.dims, sizeof(dims));
        return record_shape_op(c, LT_OP_RESHAPE, src, NONE, 0, 0, cur.rank, dims, out_node);
    }
    if (t.view_op == LT_OP_NARROW) return record_shape_op(c, LT_OP_NARROW, src, NONE, t.view_a0, t.view_a1, (int)cur.dims[t.view_a0], nullptr, out_node);
    return record_shape_op(c, LT_OP_PERMUTE, src, NONE, t.view_a0, 0, 0, nullptr, out_node);
}

// A view follows its base: if the base has been updated in place since the view's computation was derived, derive
// it again from the base's current computation (the base is brought up to date first when it is a view itself).
static lt_status sync_view(lt_ctx *c, uint32_t slot) {
    TensorRec &t0 = c->tensors[slot];
    if (t0.view_base == NONE) return LT_OK;
    if (!view_base_alive(c, t0)) {
        t0.view_base = NONE;  // the base is gone: a tensor of its own from here on
        return LT_OK;
    }
    const uint32_t b = t0.view_base;
    lt_status st = sync_view(c, b);
    if (st) return st;
    if (c->tensors[b].version == c->tensors[slot].base_seen) return LT_OK;
    uint32_t n = NONE;
    st = apply_view_op(c, c->tensors[slot], c->tensors[b].node, &n);
    if (st) return st;
    c->nodes[n].refs++;  // held across the repointing
    repoint_tensor(c, slot, n, false);
    node_unref(c, n);
    TensorRec &t = c->tensors[slot];
    t.base_seen = c->tensors[b].version;
    t.version++;
    return LT_OK;
}

// An in-place update of a view (Section 4.4): the backward sequence.  Starting from the updated value of the view,
// the inverse of each view operation gives the updated value of the next base up the chain.
static lt_status propagate_to_bases(lt_ctx *c, uint32_t slot) {
    uint32_t cur = slot;
    while (c->tensors[cur].view_base != NONE) {
        if (!view_base_alive(c, c->tensors[cur])) {
            c->tensors[cur].view_base = NONE;
            break;
        }
        const uint32_t b = c->tensors[cur].view_base;
        lt_status st = sync_view(c, b);
        if (st) return st;
        const TensorRec &t = c->tensors[cur];
        const Node base_node = c->nodes[c->tensors[b].node];
        uint32_t inv = NONE;
        if (t.view_op == LT_OP_RESHAPE) {
            int64_t dims[LT_MAX_RANK];
            memcpy(dims, base_node.dims, sizeof(dims));
            st = record_shape_op(c, LT_OP_RESHAPE, t.node, NONE, 0, 0, base_node.rank, dims, &inv);
        } else if (t.view_op == LT_OP_PERMUTE) {
            int inverse[LT_MAX_RANK] = {0};
            for (int i = 0; i < base_node.rank; ++i) inverse[(t.view_a0 >> (4 * i)) & 0xf] = i;
            st = record_shape_op(c, LT_OP_PERMUTE, t.node, NONE, (int64_t)pack_perm(inverse, base_node.rank), 0, 0, nullptr, &inv);
        } else {
            st = record_shape_op(c, LT_OP_UPDATE_SLICE, c->tensors[b].node, t.node, t.view_a0, t.view_a1, 0, nullptr, &inv);
        }
        if (st) return st;
        c->nodes[inv].refs++;
        repoint_tensor(c, b, inv, true);
        node_unref(c, inv);
        c->tensors[b].version++;
        c->tensors[cur].base_seen = c->tensors[b].version;  // this view is what the base was updated from
        cur = b;
    }
    return LT_OK;
}

static lt_status make_view(lt_ctx *c, lt_tensor t, int opcode, int64_t a0, int64_t a1, int rank, const int64_t *dims, lt_tensor *out) {
    if (!c || !out) return LT_ERR_INVALID_ARG;
    RecordTimer tm(c);
    uint32_t bs;
    trace_materialise(c);
    trace_unsupported(c);
    lt_status st = lookup(c, t, &bs);
    if (st) return st;
    uint32_t n = NONE;
    st = record_shape_op(c, opcode, c->tensors[bs].node, NONE, a0, a1, rank, dims, &n);
    if (st) return st;
    const uint32_t slot = tensor_new(c, n);
    TensorRec &v = c->tensors[slot];
    const TensorRec &b = c->tensors[bs];
    v.view_base = bs;
    v.view_base_gen = b.gen;
    v.view_op = (uint16_t)opcode;
    v.view_a0 = a0;
    v.view_a1 = a1;
    v.base_seen = b.version;
    c->view_slots.push_back(slot);
    if (c->nodes[n].op != N_DEVICE_DATA) queue_pending(c, slot);
    *out = make_handle(c, slot);
    return LT_OK;
}

}  // extern "C"
namespace {
lt_status sync_view_of(lt_ctx *c, uint32_t slot) { return sync_view(c, slot); }
}
extern "C" {

lt_status lt_op(lt_ctx *c, int opcode, const lt_tensor *in, int n_in, const int64_t *attrs, int n_attrs,
                lt_tensor *out) {
    if (!c || !out) return LT_ERR_INVALID_ARG;
    RecordTimer tm(c);
    if (c->trace.mode == TM_MATCH) {
        if (trace_match_op(c, opcode, in, n_in, attrs, n_attrs, out)) return LT_OK;
        trace_materialise(c);
    }
    if (n_in < 0 || n_in > 3 || (n_in > 0 && !in) || n_attrs < 0 || (n_attrs > 0 && !attrs))
        return fail(c, LT_ERR_INVALID_ARG, "bad operand or attribute list");
    uint32_t ids[3] = {NONE, NONE, NONE}, in_slots[3] = {NONE, NONE, NONE};
    for (int i = 0; i < n_in; ++i) {
        uint32_t slot;
        lt_status s = lookup(c, in[i], &slot);
        if (s) return s;
        in_slots[i] = slot;
        ids[i] = c->tensors[slot].node;
    }
    const Node *ops[3] = {nullptr, nullptr, nullptr};
    for (int i = 0; i < n_in; ++i) ops[i] = &c->nodes[ids[i]];

    int64_t od[LT_MAX_RANK] = {0};
    int orank = 0;
    int odtype = LT_F32;
    int64_t a0 = 0, a1 = 0;

    auto common_dtype = [&](int first, int count, int *dt) -> bool {
        int found = -1;
        for (int i = first; i < first + count; ++i)
            if (ops[i]->op != N_SCALAR) {
                if (found >= 0 && ops[i]->dtype != found) return false;
                found = ops[i]->dtype;
            }
        if (found < 0) found = ops[first]->dtype;
        for (int i = first; i < first + count; ++i)
            if (!scalar_fits(*ops[i], found)) return false;
        *dt = found;
        return true;
    };
    auto check_classes = [&](int count) -> bool {
        for (int i = 0; i < count; ++i)
            if (operand_class(*ops[i], od, orank) < 0) return false;
        return true;
    };

    if (opcode >= LT_OP_RESHAPE && opcode <= LT_OP_UPDATE_SLICE) {
        if (n_in < 1) return fail(c, LT_ERR_INVALID_ARG, std::string(op_name(opcode)) + ": wrong number of inputs or attributes");
        const Node &src = c->nodes[ids[0]];
        int64_t a0 = 0, a1 = 0;
        int rank = 0;
        const int64_t *dims = nullptr;
        bool ok = false;
        if (opcode == LT_OP_RESHAPE) {
            ok = n_in == 1 && n_attrs >= 1 && attrs[0] >= 0 && attrs[0] <= LT_MAX_RANK && n_attrs == 1 + attrs[0];
            if (ok) rank = (int)attrs[0], dims = attrs + 1;
        } else if (opcode == LT_OP_NARROW) {
            ok = n_in == 1 && n_attrs == 3 && attrs[2] <= 0x7fffffffLL;
            if (ok) a0 = attrs[0], a1 = attrs[1], rank = (int)attrs[2];
        } else if (opcode == LT_OP_PERMUTE) {
            ok = n_in == 1 && n_attrs == src.rank;
            if (ok) {
                int perm[LT_MAX_RANK];
                for (int i = 0; i < n_attrs; ++i) {
                    if (attrs[i] < 0 || attrs[i] >= src.rank) return fail(c, LT_ERR_INVALID_ARG, "permute: not a permutation of the dimensions");
                    perm[i] = (int)attrs[i];
                }
                a0 = (int64_t)pack_perm(perm, n_attrs);
            }
        } else {
            ok = n_in == 2 && n_attrs == 2;
            if (ok) a0 = attrs[0], a1 = attrs[1];
        }
        if (!ok) return fail(c, LT_ERR_INVALID_ARG, std::string(op_name(opcode)) + ": wrong number of inputs or attributes");
        uint32_t n = NONE;
        lt_status st = record_shape_op(c, opcode, ids[0], ids[1], a0, a1, rank, dims, &n);
        if (st) return st;
        const uint32_t slot = tensor_new(c, n);
        trace_unsupported(c);  // shape operations are not logged
        if (c->nodes[n].op != N_DEVICE_DATA) queue_pending(c, slot);
        *out = make_handle(c, slot);
        return LT_OK;
    }
    const bool is_binary = opcode >= LT_OP_ADD && opcode <= LT_OP_XOR;
    const bool is_compare = opcode >= LT_OP_GT && opcode <= LT_OP_NE;
    const bool is_unary = opcode >= LT_OP_NEG && opcode <= LT_OP_NOT;
    const bool is_reduce = opcode >= LT_OP_ROW_SUM && opcode <= LT_OP_ROW_MIN;
    const bool is_col_reduce = opcode >= LT_OP_COL_SUM && opcode <= LT_OP_COL_MIN;
    const bool is_all_reduce = opcode >= LT_OP_ALL_SUM && opcode <= LT_OP_ALL_MIN;

    if (is_binary || is_compare) {
        if (n_in != 2) return fail(c, LT_ERR_INVALID_ARG, "binary op takes 2 inputs");
        int dt;
        if (!common_dtype(0, 2, &dt)) return fail(c, LT_ERR_DTYPE, "operands must share one dtype");
        if (!broadcast_shape(ops, 2, od, &orank) || !check_classes(2))
            return fail(c, LT_ERR_SHAPE, "operand shapes are not a supported broadcast");
        if (is_binary) {
            bool ok;
            if (float_dtype(dt)) ok = opcode <= LT_OP_MIN;
            else if (dt == LT_U8) ok = opcode >= LT_OP_AND;
            else ok = opcode != LT_OP_DIV;
            if (!ok) return fail(c, LT_ERR_DTYPE, std::string(op_name(opcode)) + " is not defined for " + dtype_name(dt));
            odtype = dt;
        } else {
            odtype = LT_U8;
        }
    } else if (opcode == LT_OP_WHERE) {
        if (n_in != 3) return fail(c, LT_ERR_INVALID_ARG, "where takes 3 inputs");
        if (ops[0]->dtype != LT_U8 || ops[0]->op == N_SCALAR) return fail(c, LT_ERR_DTYPE, "where mask must be a u8 tensor");
        int dt;
        if (!common_dtype(1, 2, &dt)) return fail(c, LT_ERR_DTYPE, "where branches must share one dtype");
        if (!broadcast_shape(ops, 3, od, &orank) || !check_classes(3))
            return fail(c, LT_ERR_SHAPE, "operand shapes are not a supported broadcast");
        odtype = dt;
    } else if (is_unary) {
        if (n_in != 1) return fail(c, LT_ERR_INVALID_ARG, "unary op takes 1 input");
        int dt = ops[0]->dtype;
        bool ok;
        if (opcode == LT_OP_NOT) ok = dt == LT_U8;
        else if (dt == LT_I32) ok = opcode == LT_OP_NEG || opcode == LT_OP_ABS;
        else ok = float_dtype(dt);
        if (!ok) return fail(c, LT_ERR_DTYPE, std::string(op_name(opcode)) + " is not defined for " + dtype_name(dt));
        orank = ops[0]->rank;
        memcpy(od, ops[0]->dims, sizeof(od));
        odtype = dt;
    } else if (opcode == LT_OP_CONVERT) {
        if (n_in != 1 || n_attrs != 1) return fail(c, LT_ERR_INVALID_ARG, "convert takes 1 input and attrs {dtype}");
        int si = ops[0]->dtype, so = (int)attrs[0];
        if (!valid_dtype(so)) return fail(c, LT_ERR_DTYPE, "unknown target dtype");
        bool ok = (float_dtype(si) && float_dtype(so)) || (so == LT_F32 && !float_dtype(si)) ||
                  (si == LT_F32 && so == LT_I32) || (si == LT_U8 && (so == LT_I32 || so == LT_U32)) ||
                  ((si == LT_I32 || si == LT_U32) && (so == LT_I32 || so == LT_U32)) ||
                  (so == LT_U8 && si != LT_BF16);
        if (!ok) return fail(c, LT_ERR_DTYPE, std::string("convert ") + dtype_name(si) + " -> " + dtype_name(so) + " is not defined");
        orank = ops[0]->rank;
        memcpy(od, ops[0]->dims, sizeof(od));
        odtype = so;
        a0 = so;
    } else if (opcode == LT_OP_IOTA || opcode == LT_OP_PHILOX_BITS) {
        const int head = opcode == LT_OP_IOTA ? 1 : 2;
        if (n_in != 0 || n_attrs < head + 1) return fail(c, LT_ERR_INVALID_ARG, "factory op takes no inputs and attrs {.., rank, dims}");
        int r = (int)attrs[head];
        if (r < 1 || r > LT_MAX_RANK || n_attrs != head + 1 + r) return fail(c, LT_ERR_INVALID_ARG, "bad rank in attrs");
        lt_status s = check_shape(c, r, attrs + head + 1);
        if (s) return s;
        orank = r;
        for (int i = 0; i < r; ++i) od[i] = attrs[head + 1 + i];
        if (opcode == LT_OP_IOTA) {
            if (attrs[0] < 0 || attrs[0] >= r) return fail(c, LT_ERR_INVALID_ARG, "iota dim out of range");
            if (od[attrs[0]] > 2147483647LL) return fail(c, LT_ERR_UNSUPPORTED, "iota extent exceeds int32");
            odtype = LT_I32;
            a0 = attrs[0];
        } else {
            odtype = LT_U32;
            a0 = attrs[0];
            a1 = attrs[1];
        }
    } else if (is_reduce) {
        if (n_in != 1) return fail(c, LT_ERR_INVALID_ARG, "reduction takes 1 input");
        if (!float_dtype(ops[0]->dtype)) return fail(c, LT_ERR_DTYPE, "row reductions need a float dtype");
        if (ops[0]->rank < 1) return fail(c, LT_ERR_SHAPE, "row reduction needs rank >= 1");
        orank = ops[0]->rank;
        memcpy(od, ops[0]->dims, sizeof(od));
        od[orank - 1] = 1;
        odtype = ops[0]->dtype;
    } else if (is_col_reduce || is_all_reduce) {
        if (n_in != 1) return fail(c, LT_ERR_INVALID_ARG, "reduction takes 1 input");
        if (ops[0]->op == N_SCALAR) return fail(c, LT_ERR_INVALID_ARG, "reduction of a constant");
        if (!float_dtype(ops[0]->dtype)) return fail(c, LT_ERR_DTYPE, "reductions need a float dtype");
        if (is_col_reduce) {
            if (ops[0]->rank < 1) return fail(c, LT_ERR_SHAPE, "column reduction needs rank >= 1");
            orank = ops[0]->rank;
            for (int i = 0; i + 1 < orank; ++i) od[i] = 1;
            od[orank - 1] = ops[0]->dims[orank - 1];
        } else {
            orank = 0;
        }
        odtype = ops[0]->dtype;
    } else {
        return fail(c, LT_ERR_UNSUPPORTED, "unknown opcode " + std::to_string(opcode));
    }

    uint32_t n = node_new(c);  // may grow the arena: `ops` pointers are dead from here on
    Node &nd = c->nodes[n];
    nd.op = (uint16_t)opcode;
    nd.dtype = (uint8_t)odtype;
    nd.rank = (uint8_t)orank;
    nd.n_in = (uint8_t)n_in;
    for (int i = 0; i < orank; ++i) nd.dims[i] = od[i];
    nd.attr[0] = a0;
    nd.attr[1] = a1;
    for (int i = 0; i < n_in; ++i) {
        nd.in[i] = ids[i];
        node_ref(c, ids[i]);
    }
    c->stats.nodes_recorded++;
    uint32_t slot = tensor_new(c, n);
    queue_pending(c, slot);
    if (trace_learning(c)) {
        trace_log_op(c, opcode, in_slots, n_in, attrs, n_attrs, slot);
        c->trace.bind_slot.push_back(slot);
    }
    *out = make_handle(c, slot);
    return LT_OK;
}

lt_status lt_assign(lt_ctx *c, lt_tensor dst, lt_tensor src) {
    if (!c) return LT_ERR_INVALID_ARG;
    RecordTimer tm(c);
    if (c->trace.mode == TM_MATCH) {
        if (trace_match_assign(c, dst, src)) return LT_OK;
        trace_materialise(c);
    }
    uint32_t ds, ss;
    lt_status s = lookup(c, dst, &ds);
    if (s) return s;
    s = lookup(c, src, &ss);
    if (s) return s;
    TensorRec &d = c->tensors[ds];
    const TensorRec &sr = c->tensors[ss];
    if (d.view_base != NONE || sr.view_base != NONE) trace_unsupported(c);
    if (trace_learning(c)) {
        trace_log_pair(c, TE_ASSIGN, ds, ss);
        c->trace.bind_slot.push_back(NONE);
    }
    if (d.node == sr.node) return LT_OK;
    const Node &dn = c->nodes[d.node];
    const Node &sn = c->nodes[sr.node];
    bool same = dn.dtype == sn.dtype && dn.rank == sn.rank;
    for (int i = 0; same && i < dn.rank; ++i) same = dn.dims[i] == sn.dims[i];
    if (!same) return fail(c, LT_ERR_SHAPE, "lt_assign needs equal shape and dtype");
    // Section 4.3: the destination's computation is replaced by the source's; the buffer it
    // named is remembered so the barrier can write the new value in place.
    repoint_tensor(c, ds, sr.node, true);
    c->tensors[ds].version++;
    // Section 4.4: an update of a view also updates what it is a view of
    if (c->tensors[ds].view_base != NONE) return propagate_to_bases(c, ds);
    return LT_OK;
}

lt_status lt_view_reshape(lt_ctx *c, lt_tensor t, int rank, const int64_t *shape, lt_tensor *out) {
    return make_view(c, t, LT_OP_RESHAPE, 0, 0, rank, shape, out);
}

lt_status lt_view_narrow(lt_ctx *c, lt_tensor t, int dim, int64_t start, int64_t length, lt_tensor *out) {
    if (length < 1 || length > 0x7fffffffLL) return c ? fail(c, LT_ERR_SHAPE, "narrow: slice outside the dimension") : LT_ERR_INVALID_ARG;
    return make_view(c, t, LT_OP_NARROW, dim, start, (int)length, nullptr, out);
}

lt_status lt_view_permute(lt_ctx *c, lt_tensor t, const int *perm, lt_tensor *out) {
    if (!c || !perm) return LT_ERR_INVALID_ARG;
    uint32_t bs;
    lt_status st = lookup(c, t, &bs);
    if (st) return st;
    const int rank = c->nodes[c->tensors[bs].node].rank;
    for (int i = 0; i < rank; ++i)
        if (perm[i] < 0 || perm[i] >= rank) return fail(c, LT_ERR_INVALID_ARG, "permute: not a permutation of the dimensions");
    return make_view(c, t, LT_OP_PERMUTE, (int64_t)pack_perm(perm, rank), 0, 0, nullptr, out);
}

lt_status lt_release(lt_ctx *c, lt_tensor t) {
    if (!c) return LT_ERR_INVALID_ARG;
    RecordTimer tm(c);
    if (c->trace.mode == TM_MATCH) {
        if (trace_match_release(c, t)) return LT_OK;
        trace_materialise(c);
    }
    uint32_t slot;
    lt_status s = lookup(c, t, &slot);
    if (s) return s;
    if (c->tensors[slot].view_base != NONE) trace_unsupported(c);
    if (trace_learning(c)) {
        trace_log_pair(c, TE_RELEASE, slot, NONE);
        c->trace.bind_slot.push_back(NONE);
    }
    TensorRec &tr = c->tensors[slot];
    tr.live = false;
    tr.queued = false;
    if (tr.donor != NONE) {
        buffer_unref(c, tr.donor);
        tr.donor = NONE;
    }
    c->nodes[tr.node].tensor_refs--;
    node_unref(c, tr.node);
    tr.node = NONE;
    c->free_tensors.push_back(slot);
    return LT_OK;
}

lt_status lt_release_many(lt_ctx *c, const lt_tensor *handles, size_t n) {
    if (!c || (n && !handles)) return LT_ERR_INVALID_ARG;
    for (size_t i = 0; i < n; ++i) {
        lt_status s = lt_release(c, handles[i]);
        if (s) return s;
    }
    return LT_OK;
}

lt_status lt_op_many(lt_ctx *c, const lt_batch_op *ops, size_t n_ops, const lt_tensor *inputs, size_t n_inputs, const int64_t *attrs,
                     lt_tensor *results) {
    if (!c || (n_ops && (!ops || !results)) || (n_inputs && !inputs)) return LT_ERR_INVALID_ARG;
    for (size_t k = 0; k < n_ops; ++k) results[k] = 0;
    lt_status st = LT_OK;
    size_t done = 0;
    for (; done < n_ops && st == LT_OK; ++done) {
        const lt_batch_op &o = ops[done];
        const int want = o.opcode == LT_BATCH_ASSIGN ? 2 : o.n_in;
        lt_tensor in[3] = {0, 0, 0};
        if (want < 0 || want > 3 || o.n_attrs < 0 || (o.n_attrs > 0 && !attrs)) st = fail(c, LT_ERR_INVALID_ARG, "lt_op_many: bad operand or attribute count");
        for (int i = 0; i < want && st == LT_OK; ++i) {
            const int64_t r = o.in[i];
            if (r >= 0 && (size_t)r < n_inputs) in[i] = inputs[r];
            else if (r < 0 && (size_t)(-(r + 1)) < done && results[-(r + 1)]) in[i] = results[-(r + 1)];
            else st = fail(c, LT_ERR_INVALID_ARG, "lt_op_many: an operand names neither an input nor an earlier result of the batch");
        }
        if (st != LT_OK) break;
        if (o.opcode == LT_BATCH_ASSIGN) st = lt_assign(c, in[0], in[1]);
        else st = lt_op(c, o.opcode, in, o.n_in, o.n_attrs ? attrs + o.attr_offset : nullptr, o.n_attrs, &results[done]);
        if (st != LT_OK) break;
    }
    // the temporaries go, in order; after an error so does everything the batch made
    for (size_t k = 0; k < n_ops; ++k) {
        if (!results[k] || (st == LT_OK && ops[k].keep)) continue;
        const lt_status r = lt_release(c, results[k]);
        results[k] = 0;
        if (st == LT_OK && r != LT_OK) st = r;
    }
    return st;
}

lt_status lt_barrier(lt_ctx *c, int blocking) {
    if (!c) return LT_ERR_INVALID_ARG;
    DeviceScope on_device(c->device);
    if (!on_device.ok()) return fail(c, LT_ERR_CUDA, "cudaSetDevice failed for the context's device");
    if (c->trace.mode == TM_MATCH && c->trace.cursor) {
        lt_status matched = LT_OK;
        if (trace_barrier(c, blocking, &matched)) return matched;
        trace_materialise(c);
    }
    std::vector<uint32_t> &roots = c->roots_scratch;
    Canonical &cg = c->canon;
    if (!c->view_slots.empty()) {
        // live views catch up with in-place updates of their bases before the graph is closed
        size_t w = 0;
        for (size_t k = 0; k < c->view_slots.size(); ++k) {
            const uint32_t slot = c->view_slots[k];
            if (slot >= c->tensors.size() || !c->tensors[slot].live || c->tensors[slot].view_base == NONE) continue;
            lt_status st = sync_view_of(c, slot);
            if (st) return st;
            if (c->tensors[slot].view_base != NONE) c->view_slots[w++] = slot;
        }
        c->view_slots.resize(w);
    }
    {
        Timer tm(c->stats.ns_canonicalise);
        gather_roots(c, roots, false);
        if (!roots.empty()) canonicalise(c, roots, cg);
    }
    if (roots.empty()) {
        gather_roots(c, roots, true);
        if (blocking && c->device != LT_DEVICE_NONE) {
            lt_status st = sync_and_check(c);
            if (st) return st;
        }
        return LT_OK;
    }
    c->stats.barriers++;
    const uint64_t hits_before = c->stats.cache_hits;
    Plan *plan = nullptr;
    {
        Timer tm(c->stats.ns_hash_lookup);
        hash_bytes(cg.bytes.data(), cg.bytes.size(), cg.hash);
        HashKey key{{cg.hash[0], cg.hash[1]}};
        auto it = c->cache.find(key);
        if (it != c->cache.end()) {
            Plan *p = it->second.get();
            if (!c->opt.verify ||
                (p->canon_bytes.size() == cg.bytes.size() && !memcmp(p->canon_bytes.data(), cg.bytes.data(), cg.bytes.size())))
                plan = p;
            else {
                if (c->replay.plan == p) c->replay.plan = c->replay.exec = nullptr;
                trace_forget_plan(c, p);
                c->cache.erase(it);  // a colliding entry: replace it below
            }
        }
    }
    if (plan) {
        c->stats.cache_hits++;
    } else {
        Timer tm(c->stats.ns_plan);
        std::unique_ptr<Plan> np(new Plan());
        lt_status s = build_plan(c, cg, *np);
        if (s) return s;  // pending graph untouched
        np->hash[0] = cg.hash[0];
        np->hash[1] = cg.hash[1];
        np->canon_bytes = cg.bytes;
        c->stats.compiles++;
        if (c->opt.cache_capacity > 0 && (int64_t)c->cache.size() >= c->opt.cache_capacity) {
            auto victim = c->cache.begin();
            for (auto it = c->cache.begin(); it != c->cache.end(); ++it)
                if (it->second->last_used < victim->second->last_used) victim = it;
            if (c->last_plan == victim->second.get()) {
                c->last_plan_text = describe_plan(*c->last_plan);
                c->last_plan = nullptr;
            }
            if (c->replay.plan == victim->second.get()) c->replay.plan = c->replay.exec = nullptr;
            trace_forget_plan(c, victim->second.get());
            c->cache.erase(victim);
        }
        plan = np.get();
        c->cache[HashKey{{cg.hash[0], cg.hash[1]}}] = std::move(np);
    }
    plan->last_used = ++c->use_clock;
    c->last_plan = plan;
    const bool was_hit = c->stats.cache_hits != hits_before;
    if (c->opt.log >= 2 || (c->opt.log >= 1 && !was_hit)) {
        size_t compiled = 0;
        for (const Launch &L : plan->launches) compiled += L.compiled >= 0 ? 1 : 0;
        fprintf(stderr, "[lazytensor] barrier %llu: %zu nodes, hash %016llx%016llx, %s, %zu launches (%zu with a compiled kernel), %zu outputs, %zu temporaries\n",
                (unsigned long long)c->stats.barriers, cg.nodes.size(), (unsigned long long)cg.hash[0], (unsigned long long)cg.hash[1],
                was_hit ? "cache hit" : "planned", plan->launches.size(), compiled, plan->outputs.size(), plan->temp_bytes.size());
    }
    Plan *ran = plan;  // the cached plan, or its split variant when that is what this flush needed
    {
        Timer tm(c->stats.ns_bind_launch);
        lt_status s = run_plan(c, plan, cg, &ran);
        if (s) return s;  // nothing was rebound: the graph can be flushed again
    }
    {
        Timer tm(c->stats.ns_rebind);
        // Roots become device-data leaves over their output buffers; the IR behind them is dropped.
        const size_t n_out = cg.outputs.size();
        std::vector<uint32_t> new_nodes(n_out);
        for (size_t k = 0; k < n_out; ++k) {
            const OutputPlan &op = ran->outputs[k];
            uint32_t n = node_new(c);
            Node &nd = c->nodes[n];
            nd.op = N_DEVICE_DATA;
            nd.dtype = op.dtype;
            nd.rank = op.rank;
            memcpy(nd.dims, op.dims, sizeof(nd.dims));
            if (op.donated_param >= 0) {
                uint32_t b = c->nodes[cg.param_node[op.donated_param]].buffer;
                c->buffers[b].refs++;
                nd.buffer = b;
            } else {
                nd.buffer = buffer_new(c, c->out_ptr[k], op.bytes, true);
            }
            nd.refs = 1;  // held by this loop until the tensors are repointed
            new_nodes[k] = n;
        }
        consume_pending(c);  // `roots` still holds what the first pass gathered: nothing was recorded in between
        record_replay(c, plan, ran, cg, roots);
        const bool sealed = trace_seal(c, plan, ran, cg, roots);
        for (uint32_t slot : roots) {
            TensorRec &t = c->tensors[slot];
            const Node &old = c->nodes[t.node];
            int32_t k = cg.nodes[old.canon].output;
            uint32_t nn = new_nodes[k];
            uint32_t old_id = t.node;
            t.node = nn;
            node_ref(c, nn);
            c->nodes[nn].tensor_refs++;
            c->nodes[old_id].tensor_refs--;
            node_unref(c, old_id);
        }
        release_donors(c, roots);
        for (uint32_t n : new_nodes) node_unref(c, n);
        // the next trace is compared with this one if this one could be logged; after several traces in a row that
        // began like the logged one and then differed, a few are recorded without trying
        TraceState &T = c->trace;
        if (T.backoff) --T.backoff;
        trace_begin(c, sealed && !T.backoff ? TM_MATCH : TM_LEARN);
    }
    if (blocking && c->device != LT_DEVICE_NONE) return sync_and_check(c);
    return LT_OK;
}

lt_status lt_replay(lt_ctx *c, int blocking) {
    if (!c) return LT_ERR_INVALID_ARG;
    DeviceScope on_device(c->device);
    if (!on_device.ok()) return fail(c, LT_ERR_CUDA, "cudaSetDevice failed for the context's device");
    trace_materialise_if_started(c);
    ReplayRecord &r = c->replay;
    if (!r.plan) return fail(c, LT_ERR_INVALID_ARG, "lt_replay: no flushed graph to replay");
    if (!r.why_not.empty()) return fail(c, LT_ERR_UNSUPPORTED, "lt_replay: " + r.why_not);
    std::vector<uint32_t> &roots = c->roots_scratch;
    gather_roots(c, roots, false);
    if (!roots.empty()) return fail(c, LT_ERR_INVALID_ARG, "lt_replay: operations are pending; flush them with lt_barrier");
    Plan *plan = r.exec;
    auto live = [c](const ReplayRecord::Ref &ref) {
        return ref.slot < c->tensors.size() && c->tensors[ref.slot].live && c->tensors[ref.slot].gen == ref.gen;
    };
    // parameters: the current value of the tensors that supplied them
    Canonical &cg = c->canon;
    cg.param_node.resize(r.params.size());
    for (size_t i = 0; i < r.params.size(); ++i) {
        const ReplayRecord::ParamRef &pr = r.params[i];
        if (!live(pr)) return fail(c, LT_ERR_INVALID_ARG, "lt_replay: an input tensor of the recorded step has been released");
        const uint32_t n = c->tensors[pr.slot].node;
        const Node &nd = c->nodes[n];
        bool same = nd.op == N_DEVICE_DATA && nd.dtype == pr.dtype && nd.rank == pr.rank;
        for (int k = 0; same && k < pr.rank; ++k) same = nd.dims[k] == pr.dims[k];
        if (!same) return fail(c, LT_ERR_INVALID_ARG, "lt_replay: an input tensor no longer has the recorded dtype and shape");
        cg.param_node[i] = n;
    }
    for (const ReplayRecord::Root &root : r.roots)
        if (!live(root)) return fail(c, LT_ERR_INVALID_ARG, "lt_replay: a result tensor of the recorded step has been released");
    // in-place results: the buffer must still be named by the receiving tensor alone
    for (size_t k = 0; k < plan->outputs.size(); ++k) {
        const int32_t p = plan->outputs[k].donated_param;
        if (p < 0) continue;
        const Node &leaf = c->nodes[cg.param_node[p]];
        const bool ok = leaf.tensor_refs == 1 && c->buffers[leaf.buffer].refs == 1;
        if (!ok || !r.in_place_ok[k])
            return fail(c, LT_ERR_UNSUPPORTED, "lt_replay: an in-place result would overwrite memory another tensor names");
    }
    // run-time values: scalars from their tensors, the rest as recorded or set
    for (size_t k = 0; k < r.dyn.size(); ++k)
        if (r.dyn_scalar[k].slot != NONE && live(r.dyn_scalar[k])) {
            const Node &sn = c->nodes[c->tensors[r.dyn_scalar[k].slot].node];
            if (sn.op == N_SCALAR) r.dyn[k].d = sn.sval;
        }
    cg.dyn = r.dyn;
    r.plan->last_used = ++c->use_clock;
    c->last_plan = r.plan;
    {
        Timer tm(c->stats.ns_bind_launch);
        lt_status s = execute_plan(c, *plan, cg);
        if (s) return s;
    }
    {
        Timer tm(c->stats.ns_rebind);
        // A result written in place already lives where its tensor's leaf points (checked above: that
        // tensor alone names the buffer): nothing to rebind.  Fresh results get a new leaf.
        const size_t n_out = plan->outputs.size();
        std::vector<uint32_t> fresh(n_out, NONE);
        for (size_t k = 0; k < n_out; ++k) {
            const OutputPlan &op = plan->outputs[k];
            if (op.donated_param >= 0) continue;
            uint32_t n = node_new(c);
            Node &nd = c->nodes[n];
            nd.op = N_DEVICE_DATA;
            nd.dtype = op.dtype;
            nd.rank = op.rank;
            memcpy(nd.dims, op.dims, sizeof(nd.dims));
            nd.buffer = buffer_new(c, c->out_ptr[k], op.bytes, true);
            nd.refs = 1;
            fresh[k] = n;
        }
        for (const ReplayRecord::Root &root : r.roots) {
            const uint32_t nn = fresh[root.output];
            if (nn == NONE) continue;
            TensorRec &t = c->tensors[root.slot];
            const uint32_t old_id = t.node;
            t.node = nn;
            node_ref(c, nn);
            c->nodes[nn].tensor_refs++;
            c->nodes[old_id].tensor_refs--;
            node_unref(c, old_id);
        }
        for (uint32_t n : fresh)
            if (n != NONE) node_unref(c, n);
    }
    c->stats.replays++;
    if (c->opt.log >= 2)
        fprintf(stderr, "[lazytensor] replay %llu: %zu launches, %zu run-time slots\n", (unsigned long long)c->stats.replays,
                plan->launches.size(), r.dyn.size());
    if (blocking && c->device != LT_DEVICE_NONE) return sync_and_check(c);
    return LT_OK;
}

lt_status lt_scalar_set(lt_ctx *c, lt_tensor scalar, double value) {
    if (!c) return LT_ERR_INVALID_ARG;
    uint32_t slot;
    lt_status s = lookup(c, scalar, &slot);
    if (s) return s;
    Node &nd = c->nodes[c->tensors[slot].node];
    if (nd.op != N_SCALAR || !(nd.flags & NF_DYNAMIC))
        return fail(c, LT_ERR_INVALID_ARG, "lt_scalar_set: not a run-time scalar (0 and 1 are part of the graph; use lt_scalar_dynamic)");
    if (nd.refs != nd.tensor_refs) return fail(c, LT_ERR_INVALID_ARG, "lt_scalar_set: pending operations read this scalar; flush them first");
    nd.sval = value;
    return LT_OK;
}

lt_status lt_replay_slots(lt_ctx *c, uint32_t *n_slots) {
    if (!c || !n_slots) return LT_ERR_INVALID_ARG;
    *n_slots = c->replay.plan ? (uint32_t)c->replay.dyn.size() : 0u;
    return LT_OK;
}

lt_status lt_replay_set_slot(lt_ctx *c, uint32_t slot, int as_integer, double dvalue, int64_t ivalue) {
    if (!c) return LT_ERR_INVALID_ARG;
    if (!c->replay.plan || slot >= c->replay.dyn.size()) return fail(c, LT_ERR_INVALID_ARG, "lt_replay_set_slot: no such run-time slot");
    if (as_integer) c->replay.dyn[slot].i = ivalue;
    else c->replay.dyn[slot].d = dvalue;
    return LT_OK;
}

lt_status lt_debug_bounds_violations(lt_ctx *c, uint64_t *out) {
    if (!c || !out) return LT_ERR_INVALID_ARG;
    if (c->device == LT_DEVICE_NONE) return fail(c, LT_ERR_DEVICE, "lt_debug_bounds_violations needs a context on a CUDA device");
    DeviceScope on_device(c->device);
    unsigned long long n = 0;
    const int r = lt_compiled_bounds_violations(&n);
    if (r == 1) return fail(c, LT_ERR_UNSUPPORTED, "the library was not built with -DLT_DEBUG_BOUNDS");
    if (r != 0) {
        cudaGetLastError();
        return fail(c, LT_ERR_CUDA, "reading the bounds-violation counter failed");
    }
    *out = n;
    return LT_OK;
}

lt_status lt_debug_wait_probe(lt_ctx *c, uint64_t limit_ns) {
    if (!c) return LT_ERR_INVALID_ARG;
    if (c->device == LT_DEVICE_NONE) return fail(c, LT_ERR_DEVICE, "lt_debug_wait_probe needs a context on a CUDA device");
    DeviceScope on_device(c->device);
    cudaError_t e = lt_wait_probe_launch(limit_ns, c->stream);
    if (e != cudaSuccess) return fail(c, LT_ERR_CUDA, std::string("probe launch: ") + cudaGetErrorString(e));
    c->status_pending = true;
    return LT_OK;
}

lt_status lt_fetch(lt_ctx *c, lt_tensor t, void *host_dst, size_t nbytes) {
    if (!c) return LT_ERR_INVALID_ARG;
    uint32_t slot;
    if (c->trace.mode == TM_MATCH && c->trace.cursor && peek_slot(c, t, &slot) && (c->tensors[slot].vflags & (TV_VIRTUAL | TV_ASSIGNED))) {
        // a result of the trace being matched: flush first (the barrier may still find the trace repeated)
        lt_status b = lt_barrier(c, 1);
        if (b) return b;
    }
    lt_status s = lookup(c, t, &slot);
    if (s) return s;
    if (!host_dst && nbytes) return fail(c, LT_ERR_INVALID_ARG, "host destination is null");
    if (c->device == LT_DEVICE_NONE) return fail(c, LT_ERR_UNSUPPORTED, "context has no device");
    DeviceScope on_device(c->device);
    if (!on_device.ok()) return fail(c, LT_ERR_CUDA, "cudaSetDevice failed for the context's device");
    if (!is_leaf(c->nodes[c->tensors[slot].node])) {
        s = lt_barrier(c, 1);
        if (s) return s;
    }
    const Node &nd = c->nodes[c->tensors[slot].node];
    size_t bytes = (size_t)shape_numel(nd.dims, nd.rank) * dtype_size(nd.dtype);
    if (nbytes != bytes) return fail(c, LT_ERR_INVALID_ARG, "nbytes does not match the tensor size");
    if (nd.op == N_SCALAR) {
        double v = nd.sval;
        if (nd.dtype == LT_F32) { float f = (float)v; memcpy(host_dst, &f, 4); }
        else if (nd.dtype == LT_BF16) {
            float f = (float)v; uint32_t u; memcpy(&u, &f, 4);
            if ((u & 0x7fffffffu) > 0x7f800000u) u = (u >> 16) | 0x40u; else u = (u + 0x7fffu + ((u >> 16) & 1u)) >> 16;
            uint16_t h = (uint16_t)u; memcpy(host_dst, &h, 2);
        } else if (nd.dtype == LT_U8) { uint8_t b = (uint8_t)v; memcpy(host_dst, &b, 1); }
        else if (nd.dtype == LT_I32) { int32_t i = (int32_t)v; memcpy(host_dst, &i, 4); }
        else { uint32_t u = (uint32_t)v; memcpy(host_dst, &u, 4); }
        return LT_OK;
    }
    cudaError_t e = cudaMemcpyAsync(host_dst, c->buffers[nd.buffer].ptr, bytes, cudaMemcpyDeviceToHost, c->stream);
    if (e != cudaSuccess) return fail(c, LT_ERR_CUDA, std::string("device to host copy: ") + cudaGetErrorString(e));
    return sync_and_check(c);
}

lt_status lt_device_ptr(lt_ctx *c, lt_tensor t, void **dptr) {
    if (!c || !dptr) return LT_ERR_INVALID_ARG;
    uint32_t slot;
    lt_status s = lookup(c, t, &slot);
    if (s) return s;
    const Node &nd = c->nodes[c->tensors[slot].node];
    if (nd.op != N_DEVICE_DATA) return fail(c, LT_ERR_INVALID_ARG, "tensor is not materialised");
    *dptr = c->buffers[nd.buffer].ptr;
    return LT_OK;
}

lt_status lt_tensor_info(lt_ctx *c, lt_tensor t, int *dtype, int *rank, int64_t *shape, int *materialised) {
    if (!c) return LT_ERR_INVALID_ARG;
    uint32_t slot;
    if (c->trace.mode == TM_MATCH && c->trace.cursor && peek_slot(c, t, &slot) && c->tensors[slot].view_base == NONE) {
        // answered without turning the matched calls into IR: a result of the trace from the log, anything else from its node
        const TensorRec &tr = c->tensors[slot];
        if (tr.vflags & TV_VIRTUAL) {
            const TraceResult &res = c->trace.script.results[tr.trace_id];
            if (dtype) *dtype = res.dtype;
            if (rank) *rank = res.rank;
            if (shape) for (int i = 0; i < res.rank; ++i) shape[i] = res.dims[i];
            if (materialised) *materialised = 0;
        } else {
            const Node &nd = c->nodes[tr.node];
            if (dtype) *dtype = nd.dtype;
            if (rank) *rank = nd.rank;
            if (shape) for (int i = 0; i < nd.rank; ++i) shape[i] = nd.dims[i];
            if (materialised) *materialised = nd.op == N_DEVICE_DATA && !(tr.vflags & TV_ASSIGNED);
        }
        return LT_OK;
    }
    lt_status s = lookup(c, t, &slot);
    if (s) return s;
    const Node &nd = c->nodes[c->tensors[slot].node];
    if (dtype) *dtype = nd.dtype;
    if (rank) *rank = nd.rank;
    if (shape) for (int i = 0; i < nd.rank; ++i) shape[i] = nd.dims[i];
    if (materialised) *materialised = nd.op == N_DEVICE_DATA;
    return LT_OK;
}

lt_status lt_get_stats(lt_ctx *c, lt_stats *out) {
    if (!c || !out) return LT_ERR_INVALID_ARG;
    *out = c->stats;
    const double k = ns_per_tick();  // the time fields accumulate ticks
    for (uint64_t *f : {&out->ns_record, &out->ns_canonicalise, &out->ns_hash_lookup, &out->ns_plan, &out->ns_bind_launch, &out->ns_rebind})
        *f = (uint64_t)((double)*f * k);
    return LT_OK;
}

lt_status lt_reset_stats(lt_ctx *c) {
    if (!c) return LT_ERR_INVALID_ARG;
    c->stats = lt_stats{};
    return LT_OK;
}

lt_status lt_cache_size(lt_ctx *c, uint64_t *out) {
    if (!c || !out) return LT_ERR_INVALID_ARG;
    *out = c->cache.size();
    return LT_OK;
}

lt_status lt_set_kernel_timing(lt_ctx *c, int enable) {
    if (!c) return LT_ERR_INVALID_ARG;
    if (c->device == LT_DEVICE_NONE) return fail(c, LT_ERR_UNSUPPORTED, "context has no device");
    c->timing = enable != 0;
    return LT_OK;
}

lt_status lt_get_kernel_timing(lt_ctx *c, lt_kernel_timing *out) {
    if (!c || !out) return LT_ERR_INVALID_ARG;
    memset(out, 0, sizeof(*out));
    if (c->device == LT_DEVICE_NONE) return fail(c, LT_ERR_UNSUPPORTED, "context has no device");
    DeviceScope on_device(c->device);
    cudaError_t e = cudaStreamSynchronize(c->stream);
    if (e != cudaSuccess) return fail(c, LT_ERR_CUDA, std::string("cudaStreamSynchronize: ") + cudaGetErrorString(e));
    for (auto &t : c->timed) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, t.start, t.stop) == cudaSuccess) {
            out->launches[t.kind]++;
            out->ms[t.kind] += ms;
            out->bytes[t.kind] += t.bytes;
        }
        c->event_pool.push_back(t.start);
        c->event_pool.push_back(t.stop);
    }
    c->timed.clear();
    return LT_OK;
}

lt_status lt_dump_ir(lt_ctx *c, char *buf, size_t cap, size_t *need) {
    if (!c) return LT_ERR_INVALID_ARG;
    trace_materialise_if_started(c);
    std::vector<uint32_t> roots;
    gather_roots(c, roots, false);
    std::string s = "IR {\n";
    if (!roots.empty()) {
        Canonical cg;
        canonicalise(c, roots, cg);
        for (size_t i = 0; i < cg.nodes.size(); ++i) {
            const CNode &n = cg.nodes[i];
            s += "    %" + std::to_string(i) + " = " + shape_text(n.dtype, n.dims, n.rank) + " lt::";
            if (n.op == N_SCALAR && n.dyn >= 0) s += "scalar_data";
            else s += op_name(n.op);
            s += "(";
            for (int k = 0; k < n.n_in; ++k) {
                if (k) s += ", ";
                s += "%" + std::to_string(n.in[k]);
            }
            s += ")";
            if (n.op == N_DEVICE_DATA) s += ", device=" + (c->device == LT_DEVICE_NONE ? std::string("NONE") : "CUDA:" + std::to_string(c->device));
            if (n.op == N_SCALAR && n.dyn < 0) {
                char tmp[32];
                snprintf(tmp, sizeof(tmp), "%g", n.sval);
                s += std::string(", value=") + tmp;
            }
            if (n.op == LT_OP_CONVERT) s += std::string(", dtype=") + dtype_name((int)n.attr0);
            if (n.op == LT_OP_IOTA) s += ", dim=" + std::to_string(n.attr0);
            if (n.op == LT_OP_NARROW || n.op == LT_OP_UPDATE_SLICE) s += ", dim=" + std::to_string(n.attr0) + ", start=" + std::to_string(n.attr1);
            if (n.op == LT_OP_PERMUTE) {
                s += ", dims=(";
                for (int k = 0; k < n.rank; ++k) s += (k ? ", " : "") + std::to_string((n.attr0 >> (4 * k)) & 0xf);
                s += ")";
            }
            if (n.output >= 0) s += ", ROOT=" + std::to_string(n.output);
            s += "\n";
        }
    }
    s += "}\n";
    put_text(s, buf, cap, need);
    return LT_OK;
}

lt_status lt_dump_plan(lt_ctx *c, char *buf, size_t cap, size_t *need) {
    if (!c) return LT_ERR_INVALID_ARG;
    std::string s = c->last_plan ? describe_plan(*c->last_plan) : c->last_plan_text;
    put_text(s, buf, cap, need);
    return LT_OK;
}

}  // extern "C"
