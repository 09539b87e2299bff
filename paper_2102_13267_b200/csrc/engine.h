// Host-side data structures: IR arena (recorder), canonical program, plans and the context.
#pragma once
#include <cuda_runtime_api.h>
#include <stdint.h>

#include <memory>
#include <string>
#include <unordered_map>
#include <vector>

#include "../../include/lazytensor.h"
#include "jit.h"
#include "vm.h"

namespace lt {

constexpr uint16_t N_DEVICE_DATA = 200;  // leaf over a device buffer (Fig. 1: xla::device_data)
constexpr uint16_t N_SCALAR = 201;       // rank-0 constant (Fig. 1: prim::Constant)
constexpr uint32_t NONE = 0xffffffffu;

enum : uint8_t { NF_DYNAMIC = 1 };  // scalar is a run-time parameter (not 0/1, or forced)

// One IR node.  Nodes live in a flat arena and name operands by 32-bit index; shape and
// dtype are recorded on every node (Section 4.1).
struct Node {
    uint16_t op = 0;
    uint8_t dtype = 0, rank = 0;
    uint8_t n_in = 0, flags = 0;
    uint32_t in[3] = {NONE, NONE, NONE};
    uint32_t refs = 0;         // tensors + consumer nodes holding this node
    uint32_t tensor_refs = 0;  // tensors only
    uint32_t buffer = NONE;    // N_DEVICE_DATA
    uint32_t visit = 0;        // traversal stamp
    uint32_t canon = 0;        // canonical index within the current traversal
    int64_t dims[LT_MAX_RANK] = {0};
    double sval = 0.0;         // N_SCALAR value
    int64_t attr[2] = {0, 0};  // CONVERT: dtype; IOTA: dim; PHILOX: seed, offset
    // trace matching: where the node entered the trace numbered trace_epoch -- the event that made it, or
    // TID_IMPORT | the ordinal among the nodes from before the trace that it has read
    uint32_t trace_ref = 0, trace_epoch = 0;
};

struct Buffer {
    void *ptr = nullptr;
    size_t bytes = 0;
    uint32_t refs = 0;
    bool owned = false;
};

struct TensorRec {
    uint32_t node = NONE;
    uint32_t gen = 0;
    uint32_t donor = NONE;  // buffer the tensor named before lt_assign, kept for donation
    uint64_t seq = 0;       // creation order
    bool live = false;
    bool queued = false;    // already in the pending list
    // Views (Section 4.4): the tensor this one is a view of, the view operation, and how far it has followed the
    // base's in-place updates.
    uint32_t view_base = NONE, view_base_gen = 0;
    uint16_t view_op = 0;           // LT_OP_RESHAPE / NARROW / PERMUTE
    int64_t view_a0 = 0, view_a1 = 0;
    uint64_t version = 0;           // in-place updates this tensor has received
    uint64_t base_seen = 0;         // version of the base its current computation was derived from
    // trace matching: the tensor's id in the trace numbered trace_epoch (the event that made it, or TID_IMPORT |
    // the ordinal among the tensors from before the trace that it has touched), and what is pending for it
    uint32_t trace_id = 0, trace_epoch = 0;
    uint8_t vflags = 0;             // TV_*
};

// ---------------------------------------------------------------- canonical form
struct CNode {
    uint16_t op;
    uint8_t dtype, rank, n_in;
    uint32_t in[3];
    int64_t dims[LT_MAX_RANK];
    int32_t param;   // N_DEVICE_DATA: parameter ordinal
    int32_t dyn;     // first run-time slot (scalar: 1 slot; philox: 2 slots), else -1
    double sval;     // static scalar value
    int64_t attr0;   // CONVERT dtype / IOTA dim / NARROW, UPDATE_SLICE dim / PERMUTE packed permutation
    int64_t attr1;   // NARROW, UPDATE_SLICE start
    int32_t output;  // index in the output list, else -1
    uint32_t arena;  // arena node (not part of the hashed bytes)
};

union DynValue {
    double d;
    int64_t i;
};

struct Canonical {
    std::vector<CNode> nodes;
    std::vector<uint32_t> outputs;        // canonical index of each output node
    std::vector<int32_t> donor_param;     // per output: parameter ordinal whose buffer may be donated, or -1
    std::vector<uint32_t> param_node;     // per parameter: arena node (device-data leaf)
    std::vector<DynValue> dyn;            // run-time values of this trace
    std::vector<uint8_t> bytes;           // serialised form that is hashed and compared
    uint64_t hash[2] = {0, 0};
};

// -------------------------------------------------------------------------- plan
enum : uint8_t { ENC_F32 = 0, ENC_BF16 = 1, ENC_U8 = 2, ENC_I32 = 3, ENC_U32 = 4, ENC_LO32 = 5, ENC_HI32 = 6 };

struct Imm {
    int32_t dyn;    // run-time slot, or -1 for a static value
    double sval;    // static value (ENC_I32/U32 static values are integral)
    uint8_t enc;
    bool operator==(const Imm &o) const { return dyn == o.dyn && enc == o.enc && (dyn >= 0 || sval == o.sval); }
};

enum : uint8_t { IO_PARAM = 0, IO_OUTPUT = 1, IO_TEMP = 2 };

struct IoRef {
    uint8_t kind;
    uint8_t is_store;
    uint8_t dtype;
    uint8_t cls;
    uint32_t index;   // parameter ordinal / output index / temporary index
    uint32_t cnode;   // canonical node the slot carries
    uint32_t pitch = 0;    // LT_CLS_PITCHED: elements between rows of the buffer the slice is read from
    uint64_t offset = 0;   // elements from the start of the buffer to the operand's first element (a slice read in place)
};

enum : uint8_t { K_EW = 0, K_ROW = 1, K_MULTI = 2, K_RED = 3, K_VIEW = 4 };  // K_RED: a reduction that runs as a kernel of its own (reduce.cu); K_VIEW: a shape operation (views.cu)

struct Group {
    uint8_t kind = K_EW;
    uint8_t flavour = 1;  // 0 fast, 1 precise, 2 ieee (see launch.h)
    bool rowcol = false;
    uint64_t rows = 1, cols = 1;
    std::vector<uint32_t> members;  // native members (canonical indices), topological order
    std::vector<LtIns> ins;
    uint32_t n_pro = 0;             // leading instructions that run once per thread (loop-invariant loads)
    std::vector<IoRef> io;
    std::vector<Imm> imms;
    uint64_t bytes = 0;
    bool long_row = false;          // K_ROW with more columns than a row's thread group keeps in registers
    uint8_t red_axis = 0;           // K_RED: 0 rows, 1 columns, 2 everything
    uint8_t red_kind = 0;           // K_RED: 0 sum, 1 max, 2 min
    int32_t scratch_temp = -1;      // K_RED: temporary that holds the partial results, or -1
    bool fused_red = false;         // K_EW: up to three results are reduced over red_axis (1 or 2) into partial results instead of being stored (slot classes LT_CLS_REDUCED...)
    bool from_partials = false;     // K_RED: the first stage ran inside the elementwise kernel that computes the input
    uint16_t view_op = 0;           // K_VIEW: LT_OP_RESHAPE / NARROW / PERMUTE / UPDATE_SLICE
    uint8_t view_rank = 0;
    int64_t view_a0 = 0, view_a1 = 0;
    int64_t view_in_dims[LT_MAX_RANK] = {0}, view_out_dims[LT_MAX_RANK] = {0};  // of the (first) input and of the result
};

struct Launch {
    uint8_t kind = K_EW;
    uint8_t flavour = 1;
    std::vector<uint32_t> groups;   // one group, or the instances of a multi-tensor launch
    uint64_t bytes = 0;
    unsigned threads = LT_EW_THREADS;
    int compiled = -1;                   // entry of the ahead-of-time compiled table (compiled.h), or -1
    int compiled_blocks[4] = {0, 0, 0, 0};  // resident blocks per SM of that entry's kernels, by log2(chunks in flight); 0 = not asked yet
    // run-time specialisation (jit.h) of a program without a table entry: requested once the plan has run a few
    // times, used as soon as the machine code is ready
    std::unique_ptr<JitProgram> jit_program;  // null: not eligible
    std::shared_ptr<JitKernel> jit;
    bool jit_failed = false;
    uint32_t runs = 0;
    int cluster_max = -1;                // long rows: clusters of the cluster row kernel the device holds at once (-1 = not asked yet)
    std::unique_ptr<LtKParams> kp;       // K_EW / K_ROW parameter block (static parts prefilled)
    std::unique_ptr<LtMultiParams> mp;   // K_MULTI
};

struct OutputPlan {
    uint8_t dtype, rank;
    int64_t dims[LT_MAX_RANK];
    size_t bytes;
    int32_t donated_param;  // parameter ordinal whose buffer receives this output, or -1
};

struct Plan {
    uint64_t hash[2];
    std::vector<uint8_t> canon_bytes;
    uint32_t n_params = 0, n_dyn = 0;
    std::vector<OutputPlan> outputs;
    std::vector<size_t> temp_bytes;
    std::vector<Group> groups;
    std::vector<Launch> launches;
    uint64_t last_used = 0;
    // The same graph planned with every long row reduction as a kernel of its own: built when a fused long-row
    // launch cannot run on the pointers at hand (alignment), and used for that flush instead.
    std::unique_ptr<Plan> split;
};

struct Options {
    int64_t fusion = 1, verify = 1, fast_math = 1, horizontal = 1, cache_capacity = 0, ieee = 0, waves = 0, stage = 3;  // waves: 0 = each kernel's default (1; compiled multi-tensor 2)
    int64_t log = 0;  // 1: one line on stderr per planned graph (cache miss); 2: also per flush and replay
    int64_t pool_bytes = 4ll << 30;  // released device blocks the context keeps for reuse (0 = return every block at once)
    int64_t compiled = 1;  // use the ahead-of-time compiled kernel of a program when the table has one
    int64_t compiled_row_u = 0;  // chunks per thread in compiled row kernels (0 = one warp per row where it fits)
    int64_t compiled_depth = -1;  // staging depth of compiled row kernels (-1 = default, 0 = direct loads)
    int64_t compiled_u = 0;  // chunks in flight per thread in compiled elementwise / multi kernels (0 = default)
    int64_t specialise = 2;        // run-time specialisation: 0 off, 1 at planning time (blocking), 2 on a worker thread
    int64_t specialise_after = 3;  // ... once a plan has run this many times (mode 2)
    int64_t ignore_table = 0;      // measurements: plan as if the build-time table were empty (everything specialised or interpreted)
    int64_t long_l2_ahead = -1;  // long-row kernels: request the next row into L2 (-1 = the library's choice)
    int64_t cluster = 0;  // long rows: CTAs per cluster of the cluster row kernel (0 = the library's choice, 1 = never use it)
    int64_t trace_match = 1;  // a trace that repeats the previous one call by call is bound to that one's plan without being built (0 = off)
    int64_t cluster_vectors = -1;  // ... its column vectors in shared memory (1), in registers or re-read (0), the library's choice (-1)
};

struct HashKey {
    uint64_t h[2];
    bool operator==(const HashKey &o) const { return h[0] == o.h[0] && h[1] == o.h[1]; }
};
struct HashKeyHasher {
    size_t operator()(const HashKey &k) const { return (size_t)(k.h[0] ^ (k.h[1] * 0x9E3779B97F4A7C15ull)); }
};

// What lt_replay needs to run the last flushed graph again without recording it: the plan, and which
// tensors supplied its parameters and run-time scalars and received its results.
struct ReplayRecord {
    Plan *plan = nullptr;   // the cached plan of the flushed graph (null once evicted)
    Plan *exec = nullptr;   // what ran and runs again: `plan`, or the split variant it owns
    struct Ref {
        uint32_t slot = NONE, gen = 0;
    };
    struct ParamRef : Ref {
        uint8_t dtype = 0, rank = 0;
        int64_t dims[LT_MAX_RANK] = {0};
    };
    std::vector<ParamRef> params;   // tensor whose current value is parameter i
    std::vector<Ref> dyn_scalar;    // scalar tensor that supplies run-time slot k (slot == NONE: value stays as recorded)
    std::vector<DynValue> dyn;      // run-time values (recorded, or set since)
    struct Root : Ref {
        int32_t output = -1;
    };
    std::vector<Root> roots;        // tensors that receive the outputs
    std::vector<uint8_t> in_place_ok;  // per output written in place: 1 if the tensor receiving it is the one that supplies the buffer
    std::string why_not;            // non-empty: the last flush cannot be replayed, with the reason
};

// ---------------------------------------------------------------- trace matching
// The calls of one trace (from one barrier to the next), operands named relative to the trace, and how the plan
// that the trace was flushed with takes its inputs from them.  While the next trace repeats these calls one by one
// nothing is built -- no IR node, no canonical form, no hash: results are handles without a node ("virtual"), and the
// barrier binds the plan directly.  The first call that differs rebuilds the IR of the calls so far and recording
// continues as usual.
enum : uint8_t { TE_OP = 0, TE_SCALAR = 1, TE_ASSIGN = 2, TE_RELEASE = 3, TE_LEAF = 4 };
enum : uint8_t { TV_VIRTUAL = 1, TV_ASSIGNED = 2, TV_RELEASED = 4 };
constexpr uint32_t TID_IMPORT = 0x80000000u;

struct TraceEvent {
    uint8_t kind = 0, n_in = 0, n_attrs = 0, dtype = 0;
    uint16_t op = 0;
    uint8_t flags = 0, rank = 0;   // scalar: NF_DYNAMIC
    uint32_t in[3] = {0, 0, 0};    // tensor ids: operands (op), destination and source (assign), the tensor (release)
    uint32_t attr_off = 0;         // first of n_attrs words in TraceScript::attrs: an op's attributes as passed, a leaf's dimensions
    double sval = 0.0;             // static scalar: its value
};

struct TraceImport {               // a tensor from before the trace, at its first use in it
    uint32_t node_ordinal = 0;     // which of the distinct nodes read by the trace it names
    bool fresh_node = false;       // ... and whether it is the first to name it
    uint16_t op = 0;               // N_DEVICE_DATA or N_SCALAR
    uint8_t dtype = 0, rank = 0, flags = 0;
    int64_t dims[LT_MAX_RANK] = {0};
    double sval = 0.0;
};

struct TraceResult {               // dtype and shape of what an event made (answers lt_tensor_info while only matching)
    uint8_t dtype = 0, rank = 0;
    int64_t dims[LT_MAX_RANK] = {0};
};

struct TraceScript {
    std::vector<TraceEvent> events;
    std::vector<TraceResult> results;  // per event (unused for assign and release)
    std::vector<int64_t> attrs;
    std::vector<TraceImport> imports;
    uint32_t n_nodes = 0;
    // filled in when the trace is flushed
    Plan *plan = nullptr;
    std::vector<uint32_t> param_src;   // per parameter: TID_IMPORT | node ordinal, or the leaf event that made it
    struct DynSrc {
        uint32_t ref = 0;              // scalar or random-bits event, or TID_IMPORT | node ordinal of a run-time scalar
        uint8_t which = 0;             // random bits: 0 seed, 1 offset
    };
    std::vector<DynSrc> dyn_src;       // per run-time slot
    struct Root {
        uint32_t tid = 0;
        int32_t output = -1;
    };
    std::vector<Root> roots;           // in the order the barrier took them
    // for lt_replay after a matched flush: the tensors of ReplayRecord, as trace ids
    std::vector<uint32_t> replay_param, replay_dyn_scalar;
    std::vector<uint8_t> replay_in_place_ok;
    std::string replay_why_not;
    void clear() {
        events.clear(), results.clear(), attrs.clear(), imports.clear(), param_src.clear(), dyn_src.clear(), roots.clear();
        replay_param.clear(), replay_dyn_scalar.clear(), replay_in_place_ok.clear(), replay_why_not.clear();
        n_nodes = 0, plan = nullptr;
    }
};

enum : uint8_t { TM_OFF = 0, TM_LEARN = 1, TM_MATCH = 2 };

struct TraceState {
    uint8_t mode = TM_LEARN;
    bool log_valid = true;             // TM_LEARN: every call so far can be expressed as an event
    uint32_t epoch = 1;
    uint32_t cursor = 0;               // TM_MATCH: next event of `script`
    uint32_t n_imports = 0, n_nodes = 0;
    uint32_t force_slot = NONE;        // the next tensor made takes this slot (rebuilding a matched prefix)
    uint32_t streak = 0, backoff = 0;  // traces in a row that began like the log and then differed; traces left to record without trying
    TraceScript script;                // what TM_MATCH follows
    TraceScript log;                   // what TM_LEARN writes
    std::vector<uint32_t> bind_slot;          // per event of the current trace: slot of the tensor it made
    std::vector<uint32_t> bind_import_slot;   // per import: the tensor's slot
    std::vector<uint32_t> bind_node;          // per node ordinal: arena node
    std::vector<DynValue> bind_val, bind_val2;  // per event: run-time scalar value / seed, offset
    std::vector<uint32_t> deferred_release;   // TM_MATCH: tensors released since the trace began (slots kept until the barrier)
    std::vector<uint32_t> virtual_scalars;    // TM_MATCH: slots of the scalars made since the trace began
};

struct TimedLaunch {
    cudaEvent_t start, stop;
    uint8_t kind;
    uint64_t bytes;
};

}  // namespace lt

struct lt_ctx {
    int device = LT_DEVICE_NONE;
    cudaStream_t stream = nullptr;
    lt_allocator alloc{};
    bool has_alloc = false;
    uint16_t tag = 0;
    int sm_count = 148;
    int occ_ew = 2, occ_row = 2, occ_multi = 2;

    std::vector<lt::Node> nodes;
    std::vector<uint32_t> free_nodes;
    std::vector<lt::Buffer> buffers;
    std::vector<uint32_t> free_buffers;
    std::vector<lt::TensorRec> tensors;
    std::vector<uint32_t> free_tensors;
    std::vector<uint32_t> pending;  // tensor slots that may have pending IR
    std::vector<uint32_t> view_slots;  // tensor slots that are (or were) views
    uint64_t next_seq = 1;
    uint32_t stamp = 0;

    lt::Options opt;
    lt_stats stats{};
    uint32_t record_calls = 0;  // recording calls so far (one in eight is timed)
    std::unordered_map<lt::HashKey, std::unique_ptr<lt::Plan>, lt::HashKeyHasher> cache;
    uint64_t use_clock = 0;
    lt::Plan *last_plan = nullptr;
    std::string last_plan_text;  // dump of a plan that has since been evicted
    std::string error;

    // set only for the duration of lt_barrier_static_scratch: temporaries are carved out of this
    // fixed device range and nothing may be obtained from, or returned to, the allocator
    bool static_mode = false;
    bool static_clear = false;  // zero-fill the range on the stream once the flush has passed its checks
    void *static_base = nullptr;
    size_t static_cap = 0;

    lt::ReplayRecord replay;
    lt::TraceState trace;
    bool status_pending = false;      // a kernel with bounded device-side waits ran since the status word was last read
    int64_t wait_limit_ns = 2000000000ll;  // how long such a wait may last

    bool timing = false;
    std::vector<lt::TimedLaunch> timed;
    std::vector<cudaEvent_t> event_pool;

    // released device blocks by (rounded) size, and the size of every block obtained from the allocator
    std::unordered_map<size_t, std::vector<void *>> pool;
    std::unordered_map<void *, size_t> block_size;
    size_t pool_held = 0;

    // scratch reused across barriers
    lt::Canonical canon;
    std::vector<uint32_t> roots_scratch, stack_scratch, donor_scratch;
    std::vector<void *> param_ptr, out_ptr, temp_ptr;
    std::vector<uint32_t> buf_stamp;
    std::vector<int32_t> buf_param;
    std::vector<uint8_t> param_taken;
};

namespace lt {

// recorder (engine.cpp)
uint32_t node_new(lt_ctx *c);
void node_ref(lt_ctx *c, uint32_t n);
void node_unref(lt_ctx *c, uint32_t n);
uint32_t buffer_new(lt_ctx *c, void *ptr, size_t bytes, bool owned);
void buffer_unref(lt_ctx *c, uint32_t b);
size_t dtype_size(int dt);
const char *dtype_name(int dt);
const char *op_name(int op);
int64_t shape_numel(const int64_t *dims, int rank);
lt_status fail(lt_ctx *c, lt_status s, const std::string &msg);
void *ctx_alloc(lt_ctx *c, size_t bytes);
void pool_trim(lt_ctx *c, size_t keep_bytes);
void ctx_free(lt_ctx *c, void *p);

// Makes `device` the calling thread's current CUDA device for the scope and puts the previous one back
// afterwards: every entry point that enqueues work or touches device memory runs inside one, so a caller
// that has switched devices since lt_ctx_create still launches on the context's stream's device.
struct DeviceScope {
    int previous = -1;
    bool switched = false, good = true;
    explicit DeviceScope(int device) {
        if (device < 0) return;
        if (cudaGetDevice(&previous) != cudaSuccess) {
            good = false;
            return;
        }
        if (previous != device) {
            good = cudaSetDevice(device) == cudaSuccess;
            switched = good;
        }
    }
    ~DeviceScope() {
        if (switched) cudaSetDevice(previous);
    }
    bool ok() const { return good; }
    DeviceScope(const DeviceScope &) = delete;
    DeviceScope &operator=(const DeviceScope &) = delete;
};

// Chunks of eight elements per thread in the row shell (lt_c_row) for rows of `cpr` chunks: one warp per row where the
// row fits 32 x 8 chunks, else as few threads per row as eight chunks each allow -- except, measured on rows of 2048 to
// 4096 columns: a row that would take two warps at eight chunks per thread runs on four warps at four when its inputs
// are 4-byte elements or the program reads column vectors (LayerNorm f32 at 4096 columns 218 against 255 us), and a
// program with column vectors over 2-byte inputs keeps to four chunks per thread even where eight would fit one warp
// (the vectors then stay in registers: LayerNorm bf16 at 2048 columns 103 against 120 us, at 4096 105 against 151).
inline int row_chunks_per_thread(uint32_t cpr, bool has_vectors, bool four_byte_inputs) {
    int u = 1;
    while (u < 8 && cpr > 32u * (unsigned)u) u *= 2;
    if (u == 8 && cpr <= 512u) {
        if (cpr > 256u && (has_vectors || four_byte_inputs)) u = 4;
        else if (has_vectors && !four_byte_inputs) u = 4;
    }
    while (u < 8 && cpr > 128u * (unsigned)u) u *= 2;  // a row's group is at most one CTA of 128 threads
    return u;
}

// Long rows of up to 8 x 128 x 8 chunks run with a thread-block cluster as the row's thread group (lt_c_rowc): the
// cluster size and the chunks per thread for rows of `cpr` chunks; false when the row is too long.  As many chunks
// per thread as the row needs in the smallest cluster -- eight, or four when the program reads column vectors, which
// a thread then still keeps in registers (measured: softmax at 16384 columns 90 us in clusters of two against 97 in
// clusters of four; LayerNorm 129 us in clusters of four against 156 in clusters of two).
inline bool cluster_shape(uint32_t cpr, bool has_vectors, int64_t want_cluster, int64_t want_u, unsigned *cluster, int *u) {
    if (cpr > 8u * 128u * 8u || want_cluster == 1) return false;
    const unsigned prefer = has_vectors ? 4u : 8u;
    unsigned k = 2;
    while (k < 8 && (uint64_t)k * 128u * prefer < cpr) k *= 2;
    if (want_cluster == 2 || want_cluster == 4 || want_cluster == 8) k = (unsigned)want_cluster;
    int uu = 1;
    while (uu < 8 && (uint64_t)k * 128u * (unsigned)uu < cpr) uu *= 2;
    if ((want_u == 1 || want_u == 2 || want_u == 4 || want_u == 8) && (uint64_t)k * 128u * (unsigned)want_u >= cpr) uu = (int)want_u;
    if ((uint64_t)k * 128u * (unsigned)uu < cpr) return false;
    *cluster = k;
    *u = uu;
    return true;
}

// canonicaliser (canon.cpp)
void canonicalise(lt_ctx *c, const std::vector<uint32_t> &root_tensors, Canonical &out);
void hash_bytes(const uint8_t *data, size_t n, uint64_t out[2]);

// planner (planner.cpp)
lt_status build_plan(lt_ctx *c, const Canonical &cg, Plan &plan, bool isolate_long_rows = false);
std::string describe_plan(const Plan &plan);
int broadcast_class(const int64_t *dims, int rank, uint64_t rows, uint64_t cols);

// executor (executor.cpp)
lt_status execute_plan(lt_ctx *c, Plan &plan, const Canonical &cg, bool *needs_split = nullptr);
lt_status run_plan(lt_ctx *c, Plan *plan, const Canonical &cg, Plan **ran);
bool long_rows_runnable(lt_ctx *c, Plan &plan, const Canonical &cg);
void fastdiv_make(uint32_t d, uint32_t *mul, uint32_t *sh1, uint32_t *sh2);

}  // namespace lt
