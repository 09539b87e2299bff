/*
 * lazytensor.h -- C ABI of the fused-graph LazyTensor executor for NVIDIA B200 (sm_100a).
 *
 * The library implements the runtime half of the LazyTensor method (Suhan et al.,
 * "LazyTensor: combining eager execution with domain-specific compilers"):
 * tensor operations are recorded into an IR graph instead of being dispatched
 * (Section 3); a barrier call ends the graph, canonicalises and hashes it, looks
 * it up in a compile cache and executes it (Section 4); in-place updates are a
 * substitution of the destination's computation, with input buffers donated to
 * outputs at the barrier (Section 4.3).  Where the paper hands the graph to the
 * XLA compiler, this library cuts it into fusion groups, emits a small register
 * program per group and runs the group as one hand-written CUDA kernel: a kernel
 * instantiated at build time over the program itself when the program is in the
 * library's table of compiled programs, an interpreter of the program otherwise.
 *
 * Conventions
 *   - Every call returns an lt_status; LT_OK is 0.  A human-readable message for the
 *     last failing call on a context is available from lt_last_error().  No call
 *     throws, aborts or exits.  A failed lt_op records nothing; a failed lt_barrier
 *     leaves the pending graph in place so it can be flushed again.
 *   - "host" pointers are ordinary process memory; "device" pointers are CUDA global
 *     memory on the context's device.
 *   - A context and its tensors may be used by one thread at a time.  Calls that touch the device make the
 *     context's device current for their duration and restore the caller's; the stream given to
 *     lt_ctx_create must belong to that device.
 *   - Tensors are dense, row-major, contiguous.  Rank is at most LT_MAX_RANK.
 *   - Handles belong to the context that made them; a handle used with another
 *     context gives LT_ERR_DEVICE (Section 4.1: no implicit cross-device transfers).
 */
#ifndef LAZYTENSOR_H_
#define LAZYTENSOR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LT_MAX_RANK 6

/* One context per device: the liveness arena of Section 4 ("DeviceContextArena"). */
typedef struct lt_ctx lt_ctx;

/* Unique tensor identifier (Section 4: RegisterTensor / UnregisterTensor). 0 is never valid. */
typedef uint64_t lt_tensor;

typedef enum {
    LT_OK = 0,
    LT_ERR_INVALID_ARG = 1,   /* null pointer, unknown handle, bad rank, ...             */
    LT_ERR_SHAPE = 2,         /* operand shapes are not one of the supported broadcasts  */
    LT_ERR_DTYPE = 3,         /* dtype combination not defined for the op                */
    LT_ERR_DEVICE = 4,        /* handle of another context / device                      */
    LT_ERR_UNSUPPORTED = 5,   /* op or shape outside what the kernels implement          */
    LT_ERR_OOM = 6,           /* the allocator callback returned NULL                    */
    LT_ERR_CUDA = 7,          /* a CUDA runtime call failed (message has the CUDA text)  */
    LT_ERR_DEVICE_TIMEOUT = 8 /* a bounded device-side wait gave up: reported by the first blocking call
                                 (lt_barrier with blocking set, lt_fetch) after a long-row kernel ran out
                                 of time waiting for a copy into shared memory, or for the partial results
                                 of the other thread blocks of its cluster                                */
} lt_status;

typedef enum { LT_F32 = 0, LT_BF16 = 1, LT_U8 = 2, LT_I32 = 3, LT_U32 = 4 } lt_dtype;

/*
 * Traced operations ("IR compatible" operations, Section 3).  Arithmetic on LT_BF16
 * nodes is done in binary32 on widened operands and rounded to bf16 (ties to even).
 *
 * Broadcasting (Fig. 1 shows only scalar expansion; the classes here are the four the
 * kernels implement): an operand either has the result's shape, or is rank 0, or
 * has every dimension 1 except a last dimension equal to the result's ("column
 * vector", e.g. [C] or [1,C]), or equals the result's shape except for a last
 * dimension of 1 ("row scalar", e.g. [R,1]).  The operands need not include one of the result's shape:
 * [R,1] with [1,C] gives [R,C] (an outer product when the op is MUL).  Anything else is LT_ERR_SHAPE.
 * Operands share one dtype; a rank-0 scalar adopts the dtype of the tensor it meets.
 */
typedef enum {
    /* binary: 2 inputs.  f32/bf16: ADD..MIN; i32/u32: ADD SUB MUL MAX MIN AND OR XOR; u8: AND OR XOR */
    LT_OP_ADD = 1, LT_OP_SUB = 2, LT_OP_MUL = 3, LT_OP_DIV = 4, LT_OP_MAX = 5, LT_OP_MIN = 6,
    LT_OP_AND = 7, LT_OP_OR = 8, LT_OP_XOR = 9,
    /* compare: 2 inputs of one dtype -> LT_U8 holding 0 or 1 */
    LT_OP_GT = 10, LT_OP_GE = 11, LT_OP_LT = 12, LT_OP_LE = 13, LT_OP_EQ = 14, LT_OP_NE = 15,
    /* select: inputs (mask u8, a, b) -> mask != 0 ? a : b */
    LT_OP_WHERE = 16,
    /* unary, float dtypes (NEG and ABS also i32; NOT on u8: x == 0) */
    LT_OP_NEG = 20, LT_OP_ABS = 21, LT_OP_RELU = 22, LT_OP_EXP = 23, LT_OP_LOG = 24, LT_OP_TANH = 25,
    LT_OP_SQRT = 26, LT_OP_RSQRT = 27, LT_OP_RECIP = 28, LT_OP_SQUARE = 29, LT_OP_SIGMOID = 30,
    LT_OP_GELU_TANH = 31, /* 0.5 t (1 + tanh(sqrt(2/pi) (t + 0.044715 t^3))) */
    LT_OP_NOT = 32,
    /* type conversion: 1 input, attrs = {lt_dtype}.  f32->i32 truncates and saturates (NaN -> 0);
       anything -> u8 is (x != 0); i32 <-> u32 keeps the bits; u8 -> wider zero-extends. */
    LT_OP_CONVERT = 40,
    /* factory "range" (Section 3): 0 inputs, attrs = {dim, rank, d0, .., d(rank-1)} -> i32 coordinate along dim */
    LT_OP_IOTA = 41,
    /* factory "random" (Section 3): 0 inputs, attrs = {seed, offset, rank, d0, ..} -> u32.
       Element i is word (i mod 4) of the Philox4x32-10 block with counter
       (lo32(i/4), hi32(i/4), lo32(offset), hi32(offset)) and key (lo32(seed), hi32(seed)).
       seed and offset are run-time parameters: they do not enter the graph hash. */
    LT_OP_PHILOX_BITS = 42,
    /* reductions over the last dimension, kept with extent 1; float dtypes; rows of any length (rows of more
       than 8192 elements take a kernel that walks the row in slices, see lt_barrier) */
    LT_OP_ROW_SUM = 50, LT_OP_ROW_MAX = 51, LT_OP_ROW_MIN = 52,
    /* reductions over every dimension but the last: [d0, .., dk, C] -> [1, .., 1, C]; float dtypes */
    LT_OP_COL_SUM = 53, LT_OP_COL_MAX = 54, LT_OP_COL_MIN = 55,
    /* reductions over every element -> rank 0; float dtypes */
    LT_OP_ALL_SUM = 56, LT_OP_ALL_MAX = 57, LT_OP_ALL_MIN = 58,
    /* Shape operations as pure functions of their inputs (Section 4.4, Fig. 3: the IR has no aliasing; the view
       calls below are built from these).  Any dtype.
       RESHAPE: attrs = {rank, d0, ..}: same elements in row-major order under another shape.
       NARROW: attrs = {dim, start, length}: the slice [start, start + length) along dim.
       PERMUTE: attrs = {p0, .., p(rank-1)}: result dimension i is input dimension p_i.
       UPDATE_SLICE: 2 inputs (base, update), attrs = {dim, start}: base with the slice of update's extent along
       dim, starting at start, replaced by update -- the inverse of NARROW. */
    LT_OP_RESHAPE = 60, LT_OP_NARROW = 61, LT_OP_PERMUTE = 62, LT_OP_UPDATE_SLICE = 63
} lt_opcode;

/*
 * Device memory comes from the caller (e.g. PyTorch's caching allocator).  `alloc`
 * returns device memory of at least `nbytes`, aligned to 256 bytes, usable on `stream`
 * in stream order, or NULL.  `free` is called with a pointer `alloc` returned, after the
 * last kernel using it has been enqueued on `stream` (stream-ordered reuse is safe).
 * With a NULL lt_allocator the library uses cudaMallocAsync / cudaFreeAsync on the stream.
 */
typedef struct {
    void *(*alloc)(size_t nbytes, void *stream, void *user);
    void (*free)(void *dptr, void *stream, void *user);
    void *user;
} lt_allocator;

/* Counters since context creation or the last lt_reset_stats. Times are host nanoseconds. */
typedef struct {
    uint64_t nodes_recorded;     /* IR nodes appended by lt_op / factories                   */
    uint64_t barriers;           /* lt_barrier calls that found pending work                  */
    uint64_t compiles;           /* cache misses: graphs planned                             */
    uint64_t cache_hits;         /* barriers served from the plan cache                      */
    uint64_t kernels_launched;   /* all kernels                                              */
    uint64_t launches_elementwise, launches_row, launches_multi;
    uint64_t bytes_planned;      /* bytes the launched kernels were planned to read + write  */
    uint64_t outputs_donated;    /* outputs written into a donated input buffer              */
    uint64_t outputs_allocated;  /* outputs given fresh memory                               */
    uint64_t temporaries_allocated; /* cross-kernel intermediates given scratch memory        */
    uint64_t ns_record;          /* inside lt_op, lt_assign, lt_release and the factory calls (estimated: one call
                                    in eight is timed and counted eight times)                                */
    uint64_t ns_canonicalise;    /* root gathering + post-order serialisation                */
    uint64_t ns_hash_lookup;     /* hashing + cache probe                                    */
    uint64_t ns_plan;            /* fusion planning + program generation (misses only)       */
    uint64_t ns_bind_launch;     /* argument binding, allocation and kernel launches         */
    uint64_t ns_rebind;          /* turning roots into device-data leaves, freeing IR        */
    uint64_t launches_compiled;  /* of kernels_launched: ahead-of-time compiled programs     */
    uint64_t replays;            /* lt_replay calls that ran a plan                          */
    uint64_t launches_reduce;    /* reductions run as kernels of their own: over columns, over a whole tensor,
                                    over rows of more than 8192 elements outside a fused long-row kernel          */
    uint64_t launches_view;      /* shape operations run as copy kernels (narrow, permute, update_slice, and
                                    reshape where it is not folded into a program or a shared buffer)            */
    uint64_t programs_specialised; /* programs handed to the run-time specialiser (see the "specialise" option)    */
    uint64_t launches_specialised; /* of launches_compiled: kernels the run-time specialiser built                */
    uint64_t allocator_calls;    /* calls of the allocator's alloc and free (or cudaMallocAsync /
                                    cudaFreeAsync); 0 over a span means every block came from and
                                    went back to the context's own pool of released blocks          */
    uint64_t traces_matched;     /* of cache_hits: flushes whose trace repeated the previous one call by call and
                                    was bound to its plan without building the graph (the "trace_match" option)  */
    uint64_t traces_diverged;    /* traces that started out repeating the previous one and then differed          */
} lt_stats;

/* Device time per kernel family, measured with CUDA events when kernel timing is on. */
typedef struct {
    uint64_t launches[3];        /* 0 elementwise, 1 row-reduction, 2 multi-tensor */
    double ms[3];
    uint64_t bytes[3];           /* planned bytes of those launches */
} lt_kernel_timing;

/*
 * Context lifetime.  `device` is a CUDA device ordinal, or LT_DEVICE_NONE for a
 * record-and-plan-only context (no CUDA call is ever made; lt_barrier plans, counts
 * and rebinds but launches nothing; lt_fetch fails) used to test host logic.
 * `cuda_stream` is a cudaStream_t (NULL = default stream) on which all work is enqueued.
 * `allocator` may be NULL (see lt_allocator).  The context copies the struct.
 */
#define LT_DEVICE_NONE (-1)
lt_status lt_ctx_create(int device, void *cuda_stream, const lt_allocator *allocator, lt_ctx **out);
lt_status lt_ctx_destroy(lt_ctx *ctx);

/*
 * Options: "fusion" (1 default; 0 = one kernel per traced op, the unfused baseline),
 * "verify" (1 default: on a cache hit compare the canonical bytes, not just the hash),
 * "fast_math" (1 default: groups whose stored results are all bf16/u8 may use approximate
 * exp/tanh/rsqrt/division and fused multiply-add; groups storing f32 never do),
 * "ieee" (0 default: in groups storing f32, division, square root and reciprocal are accurate to
 * 2 ulp; 1 = correctly rounded, so that a graph of + - * / sqrt matches an op-by-op binary32
 * evaluation bit for bit, at about ten more instructions per element and op),
 * "cache_capacity" (0 = unbounded),
 * "compiled" (1 default: a launch whose program is in the table of ahead-of-time compiled programs, whose
 * pointers are 16-byte aligned and whose rows are a multiple of 8 elements runs on that kernel; 0 = always
 * interpret),
 * "specialise" (2 default: a program that has no kernel in the table and keeps being flushed gets one built at run
 * time -- the same kernels, instantiated over the program by the CUDA run-time compiler on a worker thread while the
 * interpreter keeps serving the flushes; 1 = build it when the graph is planned and wait for it; 0 = never.  Absent,
 * silently, when the run-time compiler library cannot be loaded.  With the environment variable LT_KERNEL_CACHE set to a
 * directory, the machine code is also kept there and found again by later processes.  Of several installed copies of
 * the run-time compiler the newest one whose code the driver can load is used; LT_NVRTC names a file instead.
 * LT_KERNEL_LOG set: the compiler's log, with registers and shared memory of every kernel, goes to stderr),
 * "specialise_after" (3 default:
 * flushes of a plan before mode 2 asks for the kernel),
 * "trace_match" (1 default: a trace -- the calls from one barrier to the next -- that repeats the previous trace call
 * by call, on tensors related to one another in the same way, is bound to the previous trace's plan at the barrier
 * without its graph being built, canonicalised or hashed (Section 7 of the paper: the cost of tracing again what has
 * not changed).  Values of run-time scalars, seeds, inputs and their addresses may differ; anything else that differs
 * makes the library build the graph of the calls so far after all, on the handles already returned, and go on as
 * usual.  Results, errors and the meaning of every call are the same with 0; only lt_stats.traces_matched and the time
 * differ.  A tensor released during a matched trace that the trace has read is unregistered at the barrier rather
 * than at the call),
 * "log" (0 default; 1 = one line on stderr for every graph that is planned, i.e. every cache miss; 2 = also one
 * line per flush and per replay; preset by the environment variable LT_LOG),
 * "wait_limit_ms" (2000 default: how long a long-row kernel waits for one of its asynchronous copies into shared
 * memory, or for the other thread blocks of its cluster, before it gives up, see LT_ERR_DEVICE_TIMEOUT),
 * "pool_bytes" (4 GiB default: device blocks the library has released are kept, up to this total, and reused
 * by later flushes before the allocator is asked; 0 = return every block at once).
 * fusion, fast_math, horizontal and ieee are part of the cache key; the others act at launch time.
 * Keys that start with "debug." select launch shapes for measurements (grid size in waves, chunks in flight
 * per thread, staging depth); they never change a result, are not part of the interface and may vanish.
 * Unknown key: LT_ERR_INVALID_ARG.  The environment variables LT_FUSION, LT_VERIFY,
 * LT_FAST_MATH, LT_HORIZONTAL preset the same options at context creation.
 */
lt_status lt_ctx_set_option(lt_ctx *ctx, const char *key, int64_t value);

/*
 * Factory from existing data (Section 3; the "device_data" leaves of Fig. 1).
 * lt_tensor_from_device BORROWS `dptr` (device): the caller keeps it alive and unchanged
 * while any tensor or pending graph refers to it; the library never frees it and writes
 * it only when the tensor is the destination of lt_assign (donation, Section 4.3).
 * 16-byte alignment enables 128-bit accesses; other alignments work, slower.
 * lt_tensor_from_host copies `hptr` (host) into memory from the allocator (owned by the
 * library, freed when the last tensor naming it is released); the copy is enqueued on the
 * stream and `hptr` may be reused after the call returns only if it is pageable memory
 * (for pinned memory: after the next blocking barrier or stream synchronisation).
 */
lt_status lt_tensor_from_device(lt_ctx *ctx, void *dptr, lt_dtype dtype, int rank, const int64_t *shape,
                                lt_tensor *out);
lt_status lt_tensor_from_host(lt_ctx *ctx, const void *hptr, lt_dtype dtype, int rank, const int64_t *shape,
                              lt_tensor *out);

/*
 * Rank-0 constant (Fig. 1: prim::Constant).  Section 4.1's heuristic: the values 0 and 1
 * (bit-equal to +0.0 or 1.0 as the double passed here) are encoded in the graph and its
 * hash; every other value is a run-time parameter, so graphs that differ only in such
 * values share one cache entry.  lt_scalar_dynamic forces the run-time class even for 0/1.
 * `dtype` is the dtype the scalar has when it meets no tensor; next to a tensor it adopts
 * the tensor's dtype (integer dtypes need an integral value: else LT_ERR_DTYPE at lt_op).
 */
lt_status lt_scalar(lt_ctx *ctx, double value, lt_dtype dtype, lt_tensor *out);
lt_status lt_scalar_dynamic(lt_ctx *ctx, double value, lt_dtype dtype, lt_tensor *out);

/*
 * Record one operation (Section 3: ops are buffered, not dispatched).  `in` holds `n_in`
 * handles, `attrs` holds `n_attrs` integers as the opcode requires.  Result shape and dtype
 * are inferred; nothing is launched.
 */
lt_status lt_op(lt_ctx *ctx, int opcode, const lt_tensor *in, int n_in, const int64_t *attrs, int n_attrs,
                lt_tensor *out);

/*
 * In-place update (Section 4.3): `dst` from now on denotes the computation behind `src`
 * (shape and dtype must match).  If `dst` was materialised data, its buffer becomes a
 * donation candidate: at the next barrier the new value is written into that buffer when
 * no other live tensor still names the old value and every read of the buffer is by the
 * kernel that overwrites it, at the same element index, or by an earlier kernel.
 */
lt_status lt_assign(lt_ctx *ctx, lt_tensor dst, lt_tensor src);

/*
 * Views (Section 4.4, "In-place operations on views").  The result shares its value with `t` the way a view shares
 * storage in an eager framework, although the IR has no mutation:
 *   - an in-place update of the view (lt_assign with the view as destination) records the forward sequence -- the
 *     view's new computation -- and the backward sequence: the inverse of every view operation between it and its
 *     base, applied in reverse order (RESHAPE back to the base's shape, PERMUTE with the inverse permutation,
 *     UPDATE_SLICE for NARROW), which becomes the base's new computation (Fig. 3);
 *   - an in-place update of the base is seen by its views: a view is derived again from the base's current
 *     computation the next time it is used.
 * Views of views work the same way, link by link.  Releasing the base leaves the view a tensor of its own.
 * Shapes and argument ranges as for LT_OP_RESHAPE / LT_OP_NARROW / LT_OP_PERMUTE.  Reshaping materialised data
 * shares the buffer; the other view operations copy at the next barrier.
 */
lt_status lt_view_reshape(lt_ctx *ctx, lt_tensor t, int rank, const int64_t *shape, lt_tensor *out);
lt_status lt_view_narrow(lt_ctx *ctx, lt_tensor t, int dim, int64_t start, int64_t length, lt_tensor *out);
lt_status lt_view_permute(lt_ctx *ctx, lt_tensor t, const int *perm, lt_tensor *out);

/* UnregisterTensor: the handle dies; a pending computation nobody names is never run.
   lt_release_many releases `n` handles in one call (language bindings batch the handles their
   garbage collector retires); it stops at the first invalid handle and reports it. */
lt_status lt_release(lt_ctx *ctx, lt_tensor t);
lt_status lt_release_many(lt_ctx *ctx, const lt_tensor *handles, size_t n);

/*
 * Several recording calls in one (Section 7 of the paper: the per-operation cost of tracing from a front end whose
 * own calls are expensive).  Entry k of `ops` is what one lt_op or lt_assign call would be; its operands are named by
 * index: in[i] >= 0 is inputs[in[i]], in[i] < 0 is the result of entry -(in[i] + 1) of the same batch.
 *   opcode >= 0          lt_op(opcode, operands, attrs + attr_offset, n_attrs); with `keep` non-zero the result's
 *                        handle is written to results[k] and belongs to the caller, otherwise the result is a temporary
 *                        of the batch, released when the batch has been recorded (results[k] = 0)
 *   LT_BATCH_ASSIGN      lt_assign(in[0], in[1]); no result
 * Exactly equivalent to making the calls one by one in order and then releasing the temporaries in order (the graph,
 * its hash and what trace matching sees are the same).  On an error the entries recorded so far are undone as far as
 * their results go (released) and the status of the failing call is returned; assignments already made stay.
 * `results` has n_ops entries.  Arrays are the caller's and only read during the call.
 */
#define LT_BATCH_ASSIGN (-1)
typedef struct {
    int32_t opcode;
    int32_t n_in;
    int32_t in[3];
    int32_t n_attrs;
    int32_t attr_offset;
    int32_t keep;
} lt_batch_op;
lt_status lt_op_many(lt_ctx *ctx, const lt_batch_op *ops, size_t n_ops, const lt_tensor *inputs, size_t n_inputs,
                     const int64_t *attrs, lt_tensor *results);

/*
 * Barrier (Section 4; mark_step / LazyTensorBarrier): materialise every live tensor that
 * has pending computation.  With `blocking` non-zero, return after the stream has drained.
 * Row reductions over more than 8192 columns: a group whose program has a kernel instantiated at build time
 * (softmax, LayerNorm, RMSNorm and the other listed groups), or built by the run-time specialiser (until then: as below), runs
 * fused -- up to 65536 columns with a thread-block cluster holding the row in registers, beyond that one thread block
 * per row walking it in slices -- when its inputs are 16-byte aligned and the row is a multiple of 8 elements; any other such graph runs
 * with each long reduction as a kernel of its own and the surrounding arithmetic as elementwise kernels.
 */
lt_status lt_barrier(lt_ctx *ctx, int blocking);

/*
 * Replay (Section 7, future work, proposes it: when the user can promise that a step's computation
 * stays the same from one iteration to the next, the graph only has to be built during the first one).
 * lt_replay runs the graph of the previous successful lt_barrier again -- no recording,
 * canonicalising or hashing -- as if the caller had issued the same lt_op / lt_assign
 * calls on the same tensor handles once more:
 *   - every input is the current value of the tensor that supplied it last time (for an in-place
 *     update x := f(x, ...), the value the previous flush or replay left in x);
 *   - every tensor that received a result receives the new result (in place where the previous
 *     flush wrote in place, otherwise in fresh memory; its previous value is released);
 *   - run-time scalars (lt_scalar with a value other than 0 or 1, lt_scalar_dynamic) are read again
 *     from their tensors, so lt_scalar_set changes them between replays; the other run-time slots
 *     (seed and offset of philox_bits) keep their values unless set with lt_replay_set_slot.
 * LT_ERR_INVALID_ARG if operations are pending, if there is nothing to replay, or if one of those
 * tensors has been released or no longer has the recorded shape; LT_ERR_UNSUPPORTED if an input of
 * the previous flush was not named by any tensor (nothing to read the new value from) or an in-place
 * result would now overwrite memory another tensor names.  Nothing has run in those cases: record
 * the step with lt_op and flush it with lt_barrier instead.
 */
lt_status lt_replay(lt_ctx *ctx, int blocking);

/* New value of a run-time scalar tensor (see lt_replay).  LT_ERR_INVALID_ARG for a handle that is not
 * a run-time scalar, or while pending operations read it (flush them first). */
lt_status lt_scalar_set(lt_ctx *ctx, lt_tensor scalar, double value);

/* Number of run-time slots of the graph lt_replay would run (0 if none), in canonical order: each
 * run-time scalar is one slot, each philox_bits op two (seed, offset). */
lt_status lt_replay_slots(lt_ctx *ctx, uint32_t *n_slots);

/* Sets run-time slot `slot` for the following replays: `as_integer` non-zero stores `ivalue` (64-bit
 * patterns: seeds, offsets), else `dvalue`.  A slot supplied by a live scalar tensor is read from the
 * tensor instead (use lt_scalar_set). */
lt_status lt_replay_set_slot(lt_ctx *ctx, uint32_t slot, int as_integer, double dvalue, int64_t ivalue);

/*
 * Barrier that obtains no device memory.  (The paper has no counterpart: its runtime always
 * allocates through the framework.)  For callers that cannot allocate while they run: a control
 * loop whose latency budget has no room for an allocator call that may synchronise the device, a
 * plug-in confined to buffers its host application handed it, a process started after another
 * framework claimed the rest of the GPU.  It does what lt_barrier does with the same kernels, but
 *   - values that pass from one kernel of the flush to a later one (the plan's temporaries) are
 *     placed in a static array in device memory of LT_STATIC_SCRATCH_MAX_BYTES bytes that every
 *     GPU using the library holds until the process exits; a graph whose temporaries (each
 *     rounded up to 256 bytes) need more is refused with LT_ERR_UNSUPPORTED;
 *   - every result must overwrite one of the graph's own inputs: lt_assign it to a tensor made
 *     by lt_tensor_from_device that the graph reads and that no other tensor names (the buffer
 *     is then written in place, Section 4.3 -- an in-place update such as x := f(x, ...)).  A
 *     result without such a buffer, or an input in memory the library owns
 *     (lt_tensor_from_host, a result of an earlier lt_barrier), is refused with
 *     LT_ERR_UNSUPPORTED;
 *   - neither the allocator callbacks nor cudaMalloc / cudaFree (or their Async forms) are called.
 * A refused call leaves the pending graph in place, so lt_barrier can still flush it.
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress, with
 * that device current); make that first call before starting any stream capture.
 * All calls, from all contexts on a device, share the one array, which keeps the previous call's
 * contents: two flushes that may overlap on the GPU (different streams, no ordering) race on it
 * and must be ordered by the caller.  No kernel of the library reads a temporary before writing
 * it; `clear_first` non-zero zero-fills the array on the stream before the flush all the same.
 */
#define LT_STATIC_SCRATCH_MAX_BYTES (32u << 20)
lt_status lt_barrier_static_scratch(lt_ctx *ctx, int blocking, int clear_first);

/*
 * IR-incompatible read-out (Section 3): runs a blocking barrier if `t` is pending, then
 * copies the tensor to `host_dst` (host).  `nbytes` must equal the tensor's byte size.
 */
lt_status lt_fetch(lt_ctx *ctx, lt_tensor t, void *host_dst, size_t nbytes);

/* Device pointer of a materialised tensor (LT_ERR_INVALID_ARG while it is pending). */
lt_status lt_device_ptr(lt_ctx *ctx, lt_tensor t, void **dptr);

/* Shape query; `shape` has room for LT_MAX_RANK entries; any out pointer may be NULL. */
lt_status lt_tensor_info(lt_ctx *ctx, lt_tensor t, int *dtype, int *rank, int64_t *shape, int *materialised);

lt_status lt_get_stats(lt_ctx *ctx, lt_stats *out);
lt_status lt_reset_stats(lt_ctx *ctx);

/* Number of plans in the cache. */
lt_status lt_cache_size(lt_ctx *ctx, uint64_t *out);

/*
 * Kernel timing: when enabled, every launch is bracketed by CUDA events on the stream.
 * lt_get_kernel_timing synchronises the stream, adds up the finished brackets since the
 * last call (or since enabling) and returns them.
 */
lt_status lt_set_kernel_timing(lt_ctx *ctx, int enable);
lt_status lt_get_kernel_timing(lt_ctx *ctx, lt_kernel_timing *out);

/*
 * Text dumps.  Both write at most `cap` bytes including the terminator into `buf` (may be
 * NULL with cap 0) and report the size needed in `*need`.
 * lt_dump_ir: the pending graph in the textual form of Fig. 1 ("%3 = f32[2,4] mul(%2, %1)",
 * roots marked ROOT=k).  lt_dump_plan: the plan the last barrier executed -- one block per
 * kernel launch with its family, geometry, inputs, outputs and register program.
 */
lt_status lt_dump_ir(lt_ctx *ctx, char *buf, size_t cap, size_t *need);
lt_status lt_dump_plan(lt_ctx *ctx, char *buf, size_t cap, size_t *need);

/*
 * Debug builds only (library compiled with -DLT_DEBUG_BOUNDS; the release build answers
 * LT_ERR_UNSUPPORTED): the ahead-of-time compiled kernels check every address they form against the
 * extent of the tensor it belongs to; an access that would leave it is redirected inside the buffer and
 * counted.  Returns the count since the library was loaded (0 is the only acceptable value).
 * Synchronises the device.
 */
lt_status lt_debug_bounds_violations(lt_ctx *ctx, uint64_t *out);

/*
 * Exercises the one device-side wait the library has, without touching any tensor: enqueues a one-warp kernel
 * that waits at most `limit_ns` nanoseconds for a completion nothing delivers, gives up and raises the device
 * status word.  The next blocking call on the context (lt_barrier with blocking set, lt_fetch) then returns
 * LT_ERR_DEVICE_TIMEOUT and clears the word; the context stays usable.
 */
lt_status lt_debug_wait_probe(lt_ctx *ctx, uint64_t limit_ns);

const char *lt_last_error(lt_ctx *ctx);
const char *lt_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LAZYTENSOR_H_ */
