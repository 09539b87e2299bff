// Device code of the ahead-of-time compiled programs: per-lane operations, the straight-line machine over a
// program given as a template parameter, and the shells (kernels) around it.  Included by compiled.cu, which
// instantiates it over the build-time table, and -- as text -- by the run-time specialiser (jit.cpp), which compiles
// the same shells for a program that has no table entry.  Self-contained apart from vm.h, vm_ops.cuh and pdl.cuh:
// no standard-library or toolkit header is needed, so that the run-time compiler can build it without an
// include path.
#pragma once
#include "pdl.cuh"
#include "vm.h"
#include "vm_ops.cuh"

template <int N>
struct IntTag {
    static constexpr int value = N;
};

namespace {

constexpr int V = LT_VM_V;
constexpr int NT = LT_VM_NT;
constexpr int C_THREADS = 256;     // elementwise and multi-tensor shells
constexpr int C_ROW_THREADS = 128; // row shell (or the row's group size, if larger)

// ------------------------------------------------------------------ program introspection
template <class PG>
struct Info {
    static constexpr __host__ __device__ bool is_ld(uint32_t op) { return op >= OP_LD && op < OP_LD + LT_VM_ND; }
    static constexpr __host__ __device__ bool is_f2m(uint32_t op) { return op >= OP_F2M && op < OP_F2M + F2M_COUNT; }
    // ordinal among the instructions that read a slot, or -1
    static constexpr __host__ __device__ int load_ordinal(int i) {
        int n = 0;
        for (int k = PG::n_pro; k < i; ++k)
            if (is_ld(PG::ins[k].op) || is_f2m(PG::ins[k].op)) ++n;
        return n;
    }
    static constexpr __host__ __device__ int n_loads() { return load_ordinal(PG::n_ins); }
    // slot a reserved (prologue-loaded) temporary stands for, or -1
    static constexpr __host__ __device__ int pro_slot(int t) {
        for (int k = 0; k < PG::n_pro; ++k)
            if ((int)(PG::ins[k].op - OP_LD) == t) return (int)PG::ins[k].imm;
        return -1;
    }
    // Staging layout of one pipeline stage (row shell): the full-class inputs of an iteration, load
    // ordinal by load ordinal; every thread owns U chunks of each.  Byte offset of load `ord`:
    static constexpr __host__ __device__ int chunk_bytes(int slot) { return PG::dtype[slot] == LT_ST_BF16 ? 16 : PG::dtype[slot] == LT_ST_U8 ? 8 : 32; }
    static constexpr __host__ __device__ int stage_offset(int ord, int u_count, int threads) {
        int off = 0, n = 0;
        for (int k = PG::n_pro; k < PG::n_ins; ++k)
            if (is_ld(PG::ins[k].op) || is_f2m(PG::ins[k].op)) {
                if (n == ord) return off;
                if (PG::cls[PG::ins[k].imm] == LT_CLS_FULL) off += chunk_bytes(PG::ins[k].imm) * u_count * threads;
                ++n;
            }
        return off;
    }
    static constexpr __host__ __device__ int stage_bytes(int u_count, int threads) { return stage_offset(1 << 20, u_count, threads); }
    // Programs that generate random bits are bound by integer issue, not by the wait for their inputs: the
    // staging copies would only add instructions (measured slower with the ring than with direct loads).
    static constexpr __host__ __device__ bool integer_heavy() {
        for (int k = 0; k < PG::n_ins; ++k)
            if (PG::ins[k].op == OP_PHILOX) return true;
        return false;
    }
    static constexpr __host__ __device__ bool is_red(uint32_t op) { return op >= OP_RED_SUM && op <= OP_RED_MIN; }
    // row reductions of the program: how many, how many before instruction i, and the kind (0 sum, 1 max, 2 min) of the r-th
    static constexpr __host__ __device__ int red_ordinal(int i) {
        int n = 0;
        for (int k = PG::n_pro; k < i; ++k)
            if (is_red(PG::ins[k].op)) ++n;
        return n;
    }
    static constexpr __host__ __device__ int n_reds() { return red_ordinal(PG::n_ins); }
    static constexpr __host__ __device__ int red_kind(int r) {
        int n = 0;
        for (int k = PG::n_pro; k < PG::n_ins; ++k)
            if (is_red(PG::ins[k].op)) {
                if (n == r) return (int)(PG::ins[k].op - OP_RED_SUM);
                ++n;
            }
        return 0;
    }
    // is slot s a full-class input (read by a load or a memory operand of the per-chunk program)?
    static constexpr __host__ __device__ bool full_input(int s) {
        if (PG::cls[s] != LT_CLS_FULL) return false;
        for (int k = PG::n_pro; k < PG::n_ins; ++k)
            if ((is_ld(PG::ins[k].op) || is_f2m(PG::ins[k].op)) && (int)PG::ins[k].imm == s) return true;
        return false;
    }
    static constexpr __host__ __device__ int elem_bytes(int s) { return PG::dtype[s] == LT_ST_BF16 ? 2 : PG::dtype[s] == LT_ST_U8 ? 1 : 4; }
    static constexpr __host__ __device__ int reserved_ordinal(int t) {  // position of reserved temporary t among the reserved ones
        int n = 0;
        for (int k = 0; k < t; ++k) n += pro_slot(k) >= 0 ? 1 : 0;
        return n;
    }
    static constexpr __host__ __device__ int n_reserved() {
        int n = 0;
        for (int t = 0; t < LT_VM_NT; ++t) n += pro_slot(t) >= 0 ? 1 : 0;
        return n;
    }
    // the slot whose value the program reduces instead of storing (LT_CLS_REDUCED...), or -1
    static constexpr __host__ __device__ int accum_slot() {
        for (int s = 0; s < PG::n_slots; ++s)
            if (PG::cls[s] >= LT_CLS_REDUCED) return s;
        return -1;
    }
    static constexpr __host__ __device__ int accum_axis() { return accum_slot() < 0 ? 0 : (PG::cls[accum_slot()] - LT_CLS_REDUCED) / 3; }
    // a program may reduce several values (all over the same axis): how many, the k-th one's slot, a slot's ordinal and kind
    static constexpr __host__ __device__ int n_accum() {
        int n = 0;
        for (int s = 0; s < PG::n_slots; ++s) n += PG::cls[s] >= LT_CLS_REDUCED ? 1 : 0;
        return n;
    }
    static constexpr __host__ __device__ int accum_slot_at(int k) {
        for (int s = 0; s < PG::n_slots; ++s)
            if (PG::cls[s] >= LT_CLS_REDUCED && k-- == 0) return s;
        return -1;
    }
    static constexpr __host__ __device__ int accum_ordinal(int slot) {
        int n = 0;
        for (int s = 0; s < slot; ++s) n += PG::cls[s] >= LT_CLS_REDUCED ? 1 : 0;
        return n;
    }
    static constexpr __host__ __device__ int accum_kind_of(int slot) { return (PG::cls[slot] - LT_CLS_REDUCED) % 3; }
    static constexpr __host__ __device__ bool needs_coords() {
        for (int k = 0; k < PG::n_ins; ++k) {
            const uint32_t op = PG::ins[k].op;
            if (op == OP_IOTA_COL || op == OP_IOTA_ROW) return true;
        }
        for (int s = 0; s < PG::n_slots; ++s)
            if (PG::cls[s] != LT_CLS_FULL && PG::cls[s] < LT_CLS_REDUCED) return true;
        return false;
    }
};

// ------------------------------------------------------------------ per-lane operations
template <int OP, int FLAV>
__device__ __forceinline__ float f2c(float a, float b) {
    if constexpr (OP == F2_DIV || OP == F2_RDIV) {
        const float n = OP == F2_DIV ? a : b, d = OP == F2_DIV ? b : a;
        float r;
        // fast: numerator times approximate reciprocal (what div.approx computes); written as two operations
        // so that the reciprocal of a broadcast divisor (a row sum) is formed once, not once per lane
        if constexpr (FLAV == 0) r = __fmul_rn(n, rcp_approx(d));
        else if constexpr (FLAV == 1) asm("div.full.f32 %0, %1, %2;" : "=f"(r) : "f"(n), "f"(d));
        else r = __fdiv_rn(n, d);
        return r;
    } else {
        return f2<OP, false>(a, b);
    }
}

// Two lanes at once.  Multiplications run as one packed mul.rn.f32x2 (each lane rounded separately, as
// in the scalar form).  Additions and subtractions stay scalar on purpose: ptxas 12.9 fuses a packed
// multiply that feeds a packed add into one packed fused multiply-add despite the explicit .rn on
// both (measured: results equal fmaf, not the two roundings), which would break the one-rounding-
// per-traced-op rule; a packed multiply feeding scalar adds is left alone.
template <int OP, int FLAV>
__device__ __forceinline__ void f2c_pair(float &a0, float &a1, float b0, float b1) {
    if constexpr (OP == F2_MUL) {
        uint64_t a, b, r;
        asm("mov.b64 %0, {%1, %2};" : "=l"(a) : "f"(a0), "f"(a1));
        asm("mov.b64 %0, {%1, %2};" : "=l"(b) : "f"(b0), "f"(b1));
        asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
        asm("mov.b64 {%0, %1}, %2;" : "=f"(a0), "=f"(a1) : "l"(r));
    } else {
        a0 = f2c<OP, FLAV>(a0, b0);
        a1 = f2c<OP, FLAV>(a1, b1);
    }
}

template <int OP, int FLAV>
__device__ __forceinline__ float unc(float x) {
    constexpr bool FAST = FLAV == 0;
    if constexpr (OP == OP_U_SQRT) return FLAV == 2 ? __fsqrt_rn(x) : sqrt_approx(x);
    else if constexpr (OP == OP_U_RSQRT) {
        float r;
        asm("rsqrt.approx.f32 %0, %1;" : "=f"(r) : "f"(x));
        return r;
    } else if constexpr (OP == OP_U_RECIP) {
        if constexpr (FLAV == 2) return __frcp_rn(x);
        else if constexpr (FLAV == 0) return rcp_approx(x);
        else {
            float r;
            asm("rcp.approx.f32 %0, %1;" : "=f"(r) : "f"(x));
            return r;
        }
    } else if constexpr (FAST && OP == OP_U_EXP) {
        float r;
        const float y = __fmul_rn(x, 1.4426950408889634f);
        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(y));
        return r;
    } else if constexpr (FAST && OP == OP_U_LOG) {
        float r;
        asm("lg2.approx.f32 %0, %1;" : "=f"(r) : "f"(x));
        return __fmul_rn(r, 0.6931471805599453f);
    } else if constexpr (FAST && OP == OP_U_SIGMOID) {
        float r;
        const float y = __fmul_rn(x, -1.4426950408889634f);
        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(y));
        return rcp_approx(__fadd_rn(r, 1.0f));
    } else if constexpr (FAST && OP == OP_U_GELU) {
        // 0.5 x (1 + tanh(k (x + c x^3))) with the polynomial in Horner form
        const float k = 0.7978845608028654f, kc = 0.7978845608028654f * 0.044715f;
        const float inner = __fmul_rn(fmaf(__fmul_rn(x, x), kc, k), x);
        const float h = __fmul_rn(x, 0.5f);
        return fmaf(h, tanh_approx(inner), h);
    } else {
        return un<OP, FAST>(x);
    }
}

// ------------------------------------------------------------------ chunk memory access
struct Raw {  // a chunk in storage format: 32 bytes of 4-byte elements, 16 of 2-byte, 8 of 1-byte
    uint4 a, b;
};

template <int DT>
__device__ __forceinline__ void raw_load(Raw &r, const char *p, bool streaming) {
    if constexpr (DT == LT_ST_BF16) {
        r.a = streaming ? __ldcs(reinterpret_cast<const uint4 *>(p)) : __ldg(reinterpret_cast<const uint4 *>(p));
    } else if constexpr (DT == LT_ST_U8) {
        const uint2 w = streaming ? __ldcs(reinterpret_cast<const uint2 *>(p)) : __ldg(reinterpret_cast<const uint2 *>(p));
        r.a.x = w.x;
        r.a.y = w.y;
    } else {
        const uint4 *q = reinterpret_cast<const uint4 *>(p);
        r.a = streaming ? __ldcs(q) : __ldg(q);
        r.b = streaming ? __ldcs(q + 1) : __ldg(q + 1);
    }
}

template <int DT>
__device__ __forceinline__ void raw_widen(float (&d)[V], const Raw &r) {
    if constexpr (DT == LT_ST_BF16) {
        const uint32_t w[4] = {r.a.x, r.a.y, r.a.z, r.a.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            d[2 * j] = u2f(w[j] << 16);
            d[2 * j + 1] = u2f(w[j] & 0xffff0000u);
        }
    } else if constexpr (DT == LT_ST_U8) {
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            d[b] = u2f((r.a.x >> (8 * b)) & 0xffu);
            d[4 + b] = u2f((r.a.y >> (8 * b)) & 0xffu);
        }
    } else {
        d[0] = u2f(r.a.x); d[1] = u2f(r.a.y); d[2] = u2f(r.a.z); d[3] = u2f(r.a.w);
        d[4] = u2f(r.b.x); d[5] = u2f(r.b.y); d[6] = u2f(r.b.z); d[7] = u2f(r.b.w);
    }
}

template <int DT>
__device__ __forceinline__ void chunk_store(const float (&a)[V], char *p) {
    if constexpr (DT == LT_ST_BF16) {
        uint4 w;
        w.x = pack_bf16x2(a[0], a[1]);
        w.y = pack_bf16x2(a[2], a[3]);
        w.z = pack_bf16x2(a[4], a[5]);
        w.w = pack_bf16x2(a[6], a[7]);
        __stcs(reinterpret_cast<uint4 *>(p), w);
    } else if constexpr (DT == LT_ST_U8) {
        uint2 w;
        w.x = (f2u(a[0]) & 0xffu) | ((f2u(a[1]) & 0xffu) << 8) | ((f2u(a[2]) & 0xffu) << 16) | (f2u(a[3]) << 24);
        w.y = (f2u(a[4]) & 0xffu) | ((f2u(a[5]) & 0xffu) << 8) | ((f2u(a[6]) & 0xffu) << 16) | (f2u(a[7]) << 24);
        __stcs(reinterpret_cast<uint2 *>(p), w);
    } else {
        __stcs(reinterpret_cast<uint4 *>(p), make_uint4(f2u(a[0]), f2u(a[1]), f2u(a[2]), f2u(a[3])));
        __stcs(reinterpret_cast<uint4 *>(p) + 1, make_uint4(f2u(a[4]), f2u(a[5]), f2u(a[6]), f2u(a[7])));
    }
}

// Asynchronous copies global -> shared, completion tracked per thread in commit groups.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async8(uint32_t dst, const void *src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait(uint32_t pending) {  // at most `pending` newest groups still in flight
    if (pending == 0) asm volatile("cp.async.wait_group 0;" ::: "memory");
    else if (pending == 1) asm volatile("cp.async.wait_group 1;" ::: "memory");
    else if (pending == 2) asm volatile("cp.async.wait_group 2;" ::: "memory");
    else asm volatile("cp.async.wait_group 3;" ::: "memory");
}

constexpr __host__ __device__ int esz_shift(int dt) { return dt == LT_ST_BF16 ? 1 : (dt == LT_ST_U8 ? 0 : 2); }

// Debug build (-DLT_DEBUG_BOUNDS): every address the shells form is checked against the extent of its slot;
// an access that would leave it is counted in a device word the host can read, and redirected to element 0 so
// that it stays inside the buffer.  The release build contains none of this.
#ifdef LT_DEBUG_BOUNDS
__device__ unsigned long long lt_c_bounds_violations = 0;
__device__ __forceinline__ uint64_t bounds_checked(uint64_t first, uint32_t count, uint64_t extent) {
    if (first + count > extent) {
        atomicAdd(&lt_c_bounds_violations, 1ull);
        return 0;
    }
    return first;
}
#define LT_CHECKED(first, count, extent) bounds_checked((first), (count), (extent))
#else
#define LT_CHECKED(first, count, extent) (first)
#endif

// Coordinates of the U chunks a thread works on in one iteration.
template <int U>
struct Coords {
    uint64_t flat0[U];  // flat index of lane 0
    uint32_t col0[U];   // column of lane 0
    uint32_t row[U];
    bool ok[U];         // the chunk exists
};

// No row reductions in this shell.
struct NoReduce {
    template <int KIND, int U, bool GUARD>
    __device__ __forceinline__ void operator()(float (&)[U][V], const bool (&)[U]) const {}
};

// An elementwise program whose result is reduced over columns or over everything: the thread keeps one accumulator
// per lane (a thread owns the same columns throughout, or the lanes are folded at the end).  Sums are kept in binary64
// and rounded once, when the second stage writes the result; the two chunks a thread computes per iteration are added
// in binary32 first (one conversion and one binary64 addition per two elements: the conversions, not memory, bound
// the kernel otherwise), an error of at most 2^-24 of each pair's sum, independent of how many rows there are.  Max
// and min are exact in binary32 and propagate NaN.
constexpr int C_MAX_REDUCED = 3;  // values one elementwise program may reduce

template <int KIND>
struct AccumOps {
    static __device__ __forceinline__ double comb(double x, double y) {
        if constexpr (KIND == 0) return x + y;
        else if constexpr (KIND == 1) return (x != x || y != y) ? x + y : (x > y ? x : y);
        else return (x != x || y != y) ? x + y : (x < y ? x : y);
    }
    static __device__ __forceinline__ float combf(float x, float y) {
        if constexpr (KIND == 1) return max_nan(x, y);
        else return min_nan(x, y);
    }
    static __device__ __forceinline__ double ident() { return KIND == 0 ? 0.0 : (KIND == 1 ? -(double)LT_INF : (double)LT_INF); }
};

// The accumulators of N reduced values: binary64 for sums, binary32 for max / min (only what a value's kind uses is kept).
template <int N>
struct AccumSet {
    double sum[N][V];
    float ext[N][V];
    template <int ORD, int KIND>
    __device__ __forceinline__ void reset() {
#pragma unroll
        for (int i = 0; i < V; ++i) {
            if constexpr (KIND == 0) sum[ORD][i] = 0.0;
            else ext[ORD][i] = KIND == 1 ? -LT_INF : LT_INF;
        }
    }
    template <int ORD, int KIND>
    __device__ __forceinline__ double get(int i) const {
        if constexpr (KIND == 0) return sum[ORD][i];
        else return (double)ext[ORD][i];
    }
    // the values of the thread's two chunks of this iteration (either may be absent)
    template <int ORD, int KIND>
    __device__ __forceinline__ void put(const float (&v0)[V], bool ok0, const float (&v1)[V], bool ok1) {
        if constexpr (KIND == 0) {
            if (ok0 && ok1) {
#pragma unroll
                for (int i = 0; i < V; ++i) sum[ORD][i] += (double)__fadd_rn(v0[i], v1[i]);
            } else if (ok0 || ok1) {
#pragma unroll
                for (int i = 0; i < V; ++i) sum[ORD][i] += (double)(ok0 ? v0[i] : v1[i]);
            }
        } else {
            if (ok0) {
#pragma unroll
                for (int i = 0; i < V; ++i) ext[ORD][i] = AccumOps<KIND>::combf(ext[ORD][i], v0[i]);
            }
            if (ok1) {
#pragma unroll
                for (int i = 0; i < V; ++i) ext[ORD][i] = AccumOps<KIND>::combf(ext[ORD][i], v1[i]);
            }
        }
    }
    template <int K2, int U, bool GUARD>
    __device__ __forceinline__ void operator()(float (&)[U][V], const bool (&)[U]) const {}
};

// Row reductions of a thread group of `group` threads (power of two) inside a CTA.
struct GroupReduce {
    float *smem;     // 2 x 32 floats, alternating between consecutive reductions
    uint32_t group;  // threads per row
    uint32_t phase;
    template <int KIND, int U, bool GUARD>
    __device__ __forceinline__ void operator()(float (&acc)[U][V], const bool (&ok)[U]) {
        const float ident = KIND == 0 ? 0.0f : (KIND == 1 ? -LT_INF : LT_INF);
        float part[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            // pairwise over the eight lanes, then over the chunks
            float l0 = red_comb<KIND>(acc[u][0], acc[u][1]), l1 = red_comb<KIND>(acc[u][2], acc[u][3]);
            float l2 = red_comb<KIND>(acc[u][4], acc[u][5]), l3 = red_comb<KIND>(acc[u][6], acc[u][7]);
            part[u] = (!GUARD || ok[u]) ? red_comb<KIND>(red_comb<KIND>(l0, l1), red_comb<KIND>(l2, l3)) : ident;
        }
#pragma unroll
        for (int s = 1; s < U; s <<= 1)
#pragma unroll
            for (int u = 0; u + s < U; u += 2 * s) part[u] = red_comb<KIND>(part[u], part[u + s]);
        float r = part[0];
        if (group >= 32u) {  // the usual case, a whole warp (or more) per row: five fixed butterfly steps
#pragma unroll
            for (uint32_t off = 16; off > 0; off >>= 1) r = red_comb<KIND>(r, __shfl_xor_sync(0xffffffffu, r, off));
        } else {
            for (uint32_t off = group >> 1; off > 0; off >>= 1) r = red_comb<KIND>(r, __shfl_xor_sync(0xffffffffu, r, off));
        }
        if (group > 32u) {
            float *buf = smem + (phase & 1u) * 32u;
            ++phase;
            const uint32_t warp = threadIdx.x >> 5;
            if ((threadIdx.x & 31u) == 0) buf[warp] = r;
            __syncthreads();
            const uint32_t wpr = group >> 5;
            const uint32_t first = (warp / wpr) * wpr;
            r = buf[first];
            for (uint32_t w = 1; w < wpr; ++w) r = red_comb<KIND>(r, buf[first + w]);
        }
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
            for (int i = 0; i < V; ++i) acc[u][i] = r;
    }
    template <int KIND>
    static __device__ __forceinline__ float red_comb(float a, float b) {
        if constexpr (KIND == 0) return __fadd_rn(a, b);
        else if constexpr (KIND == 1) return max_nan(a, b);
        else return min_nan(a, b);
    }
};

// ------------------------------------------------------------------ the machine
// State and straight-line execution of program PG on U chunks at once.  `Ptr` gives the base
// pointer of a slot, `Scal` the 32-bit immediates.
// GUARD false: every chunk of every iteration exists, so validity tests disappear.
template <class PG, int U, class Ptr, class Scal, class Red, bool GUARD = true, int HOISTED = 0>
struct Machine {
    using I = Info<PG>;
    static constexpr int FLAV = PG::flavour;
    static constexpr int NL = I::n_loads() > 0 ? I::n_loads() : 1;

    float acc[U][V];
    float t[NT][U][V];
    Raw raw[NL][U];  // storage-format chunks requested at the top of the iteration
    const Ptr &ptr;
    const Scal &scal;
    Red &red;
    const Coords<U> &ck;
    const float (*hoisted)[U][V] = nullptr;  // HOISTED 1: the reserved temporaries' column vectors, loaded once per thread
    const float *hoisted_shared = nullptr;   // HOISTED 2: the same in shared memory, [reserved ordinal][u][thread][V] (128-thread CTAs)

    __device__ __forceinline__ Machine(const Ptr &p, const Scal &s, Red &r, const Coords<U> &c) : ptr(p), scal(s), red(r), ck(c) {}

    template <int SLOT>
    __device__ __forceinline__ const char *address(int u) const {
        constexpr int cls = PG::cls[SLOT], sh = esz_shift(PG::dtype[SLOT]);
        const char *base = reinterpret_cast<const char *>(ptr(SLOT));
        if constexpr (cls == LT_CLS_FULL) return base + (LT_CHECKED(ck.flat0[u], V, ptr.extent(cls)) << sh);
        else if constexpr (cls == LT_CLS_PITCHED) return base + (((uint64_t)ck.row[u] * ptr.pitch(SLOT) + ck.col0[u]) << sh);
        else if constexpr (cls == LT_CLS_COLVEC) return base + (LT_CHECKED((uint64_t)ck.col0[u], V, ptr.extent(cls)) << sh);
        else if constexpr (cls == LT_CLS_ROWVEC) return base + (LT_CHECKED((uint64_t)ck.row[u], 1, ptr.extent(cls)) << sh);
        else return base;
    }

    // widened chunk of a slot read at the point of use (column vectors, broadcast elements)
    template <int SLOT>
    __device__ __forceinline__ void load_now(float (&d)[V], int u) const {
        constexpr int cls = PG::cls[SLOT], dt = PG::dtype[SLOT];
        const char *p = address<SLOT>(u);
        if constexpr (cls <= LT_CLS_COLVEC || cls == LT_CLS_PITCHED) {
            Raw r;
            raw_load<dt>(r, p, cls == LT_CLS_PITCHED);  // (a slice is streamed like any full-class operand)
            raw_widen<dt>(d, r);
        } else {
            float x;
            if constexpr (dt == LT_ST_BF16) x = u2f((uint32_t)__ldg(reinterpret_cast<const unsigned short *>(p)) << 16);
            else if constexpr (dt == LT_ST_U8) x = u2f((uint32_t)__ldg(reinterpret_cast<const unsigned char *>(p)));
            else x = __ldg(reinterpret_cast<const float *>(p));
#pragma unroll
            for (int i = 0; i < V; ++i) d[i] = x;
        }
    }

    // requests every full-class input of the iteration
    __device__ __forceinline__ void issue_loads() { request<PG::n_pro>(ptr, ck, raw); }

    // the same for the chunks `c` (this or a later iteration's), into `dst`
    template <int K = PG::n_pro>
    static __device__ __forceinline__ void request(const Ptr &ptr, const Coords<U> &c, Raw (&dst)[NL][U]) {
        if constexpr (K < PG::n_ins) {
            constexpr uint32_t op = PG::ins[K].op;
            if constexpr (I::is_ld(op) || I::is_f2m(op)) {
                constexpr int slot = PG::ins[K].imm;
                if constexpr (PG::cls[slot] == LT_CLS_FULL) {
                    constexpr int dt = PG::dtype[slot], sh = esz_shift(dt);
                    const char *base = reinterpret_cast<const char *>(ptr(slot));
#pragma unroll
                    for (int u = 0; u < U; ++u)
                        if (!GUARD || c.ok[u])
                            raw_load<dt>(dst[I::load_ordinal(K)][u], base + (LT_CHECKED(c.flat0[u], V, ptr.extent(LT_CLS_FULL)) << sh), true);
                }
            }
            request<K + 1>(ptr, c, dst);
        }
    }

    // Pipeline stage of the row shell.  stage_issue starts the asynchronous copies of an iteration's
    // full-class inputs into the stage at shared address `stage`; stage_fetch moves a landed stage into
    // the registers issue_loads would have filled.  A thread reads back only what it copied itself.
    template <int THREADS, int K = PG::n_pro>
    static __device__ __forceinline__ void stage_issue(const Ptr &ptr, const uint64_t (&flat0)[U], const bool (&ok)[U], uint32_t stage) {
        if constexpr (K < PG::n_ins) {
            constexpr uint32_t op = PG::ins[K].op;
            if constexpr (I::is_ld(op) || I::is_f2m(op)) {
                constexpr int slot = PG::ins[K].imm;
                if constexpr (PG::cls[slot] == LT_CLS_FULL) {
                    constexpr int cb = I::chunk_bytes(slot), sh = esz_shift(PG::dtype[slot]);
                    constexpr int off = I::stage_offset(I::load_ordinal(K), U, THREADS);
                    const char *base = reinterpret_cast<const char *>(ptr(slot));
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        if (GUARD && !ok[u]) continue;
                        const char *src = base + (LT_CHECKED(flat0[u], V, ptr.extent(LT_CLS_FULL)) << sh);
                        if constexpr (cb == 8) {
                            cp_async8(stage + off + (u * THREADS + threadIdx.x) * 8, src);
                        } else {
                            cp_async16(stage + off + (u * THREADS + threadIdx.x) * 16, src);
                            if constexpr (cb == 32) cp_async16(stage + off + ((U + u) * THREADS + threadIdx.x) * 16, src + 16);
                        }
                    }
                }
            }
            stage_issue<THREADS, K + 1>(ptr, flat0, ok, stage);
        }
    }

    template <int THREADS, int K = PG::n_pro>
    __device__ __forceinline__ void stage_fetch(const unsigned char *stage) {
        if constexpr (K < PG::n_ins) {
            constexpr uint32_t op = PG::ins[K].op;
            if constexpr (I::is_ld(op) || I::is_f2m(op)) {
                constexpr int slot = PG::ins[K].imm;
                if constexpr (PG::cls[slot] == LT_CLS_FULL) {
                    constexpr int cb = I::chunk_bytes(slot);
                    constexpr int ord = I::load_ordinal(K);
                    const unsigned char *b = stage + I::stage_offset(ord, U, THREADS);
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        if constexpr (cb == 8) {
                            const uint2 w = *reinterpret_cast<const uint2 *>(b + (u * THREADS + threadIdx.x) * 8);
                            raw[ord][u].a.x = w.x;
                            raw[ord][u].a.y = w.y;
                        } else {
                            raw[ord][u].a = *reinterpret_cast<const uint4 *>(b + (u * THREADS + threadIdx.x) * 16);
                            if constexpr (cb == 32) raw[ord][u].b = *reinterpret_cast<const uint4 *>(b + ((U + u) * THREADS + threadIdx.x) * 16);
                        }
                    }
                }
            }
            stage_fetch<THREADS, K + 1>(stage);
        }
    }

    // value of the slot instruction K reads, widened
    template <int K>
    __device__ __forceinline__ void operand_of(float (&d)[V], int u) const {
        constexpr int slot = PG::ins[K].imm;
        if constexpr (PG::cls[slot] == LT_CLS_FULL) {
            constexpr int dt = PG::dtype[slot];
            raw_widen<dt>(d, raw[I::load_ordinal(K)][u]);
        } else {
            load_now<slot>(d, u);
        }
    }

    // second operand of a two-operand opcode: a temporary (a reserved one is read from its column
    // vector here) or a broadcast immediate
    template <int SRC, int IMM>
    __device__ __forceinline__ void source(float (&d)[V], int u) const {
        if constexpr (SRC == LT_VM_SRC_S) {
            const float s = u2f(scal(IMM));
#pragma unroll
            for (int i = 0; i < V; ++i) d[i] = s;
        } else if constexpr (I::pro_slot(SRC) >= 0) {
            if constexpr (HOISTED == 1) {
#pragma unroll
                for (int i = 0; i < V; ++i) d[i] = hoisted[SRC][u][i];
            } else if constexpr (HOISTED == 2) {
                const float4 *q = reinterpret_cast<const float4 *>(hoisted_shared + ((I::reserved_ordinal(SRC) * U + u) * C_ROW_THREADS + threadIdx.x) * V);
                const float4 a = q[0], b = q[1];
                d[0] = a.x, d[1] = a.y, d[2] = a.z, d[3] = a.w, d[4] = b.x, d[5] = b.y, d[6] = b.z, d[7] = b.w;
            } else {
                load_now<I::pro_slot(SRC)>(d, u);
            }
        } else {
#pragma unroll
            for (int i = 0; i < V; ++i) d[i] = t[SRC][u][i];
        }
    }

    template <int K>
    __device__ __forceinline__ void step() {
        constexpr uint32_t op = PG::ins[K].op;
        constexpr uint32_t imm = PG::ins[K].imm;
        if constexpr (op >= OP_MOV_T_ACC && op < OP_MOV_T_ACC + NT) {
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int i = 0; i < V; ++i) t[op - OP_MOV_T_ACC][u][i] = acc[u][i];
        } else if constexpr (op >= OP_MOV_ACC_T && op < OP_MOV_ACC_T + NT) {
#pragma unroll
            for (int u = 0; u < U; ++u) source<op - OP_MOV_ACC_T, 0>(acc[u], u);
        } else if constexpr (op == OP_MOV_ACC_S) {
#pragma unroll
            for (int u = 0; u < U; ++u) source<LT_VM_SRC_S, imm>(acc[u], u);
        } else if constexpr (op == OP_ST) {
            static_assert(PG::cls[imm] == LT_CLS_FULL || PG::cls[imm] == LT_CLS_ROWVEC || PG::cls[imm] >= LT_CLS_REDUCED,
                          "results are full-class, one value per row, or reduced");
            if constexpr (PG::cls[imm] >= LT_CLS_REDUCED) {
                // the values, rounded as the store they replace would round them, go into the thread's accumulators
                static_assert(U == 2, "the reducing shell computes two chunks per iteration");
                constexpr bool to_bf16 = PG::dtype[imm] == LT_ST_BF16;
                float v[2][V];
#pragma unroll
                for (int u = 0; u < 2; ++u)
#pragma unroll
                    for (int i = 0; i < V; ++i) {
                        if constexpr (to_bf16) v[u][i] = round_bf16(acc[u][i]);
                        else v[u][i] = acc[u][i];
                    }
                red.template put<I::accum_ordinal(imm), I::accum_kind_of(imm)>(v[0], !GUARD || ck.ok[0], v[1], !GUARD || ck.ok[1]);
            } else if constexpr (PG::cls[imm] == LT_CLS_FULL) {
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (!GUARD || ck.ok[u]) chunk_store<PG::dtype[imm]>(acc[u], const_cast<char *>(address<imm>(u)));
            } else {
                // one value per row (a reduction's result): written by the thread that owns the row's first chunk
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if ((!GUARD || ck.ok[u]) && ck.col0[u] == 0) {
                        char *p = const_cast<char *>(address<imm>(u));
                        constexpr int dt = PG::dtype[imm];
                        if constexpr (dt == LT_ST_BF16) *reinterpret_cast<unsigned short *>(p) = (unsigned short)(f2u(round_bf16(acc[u][0])) >> 16);
                        else if constexpr (dt == LT_ST_U8) *reinterpret_cast<unsigned char *>(p) = (unsigned char)f2u(acc[u][0]);
                        else *reinterpret_cast<float *>(p) = acc[u][0];
                    }
            }
        } else if constexpr (op == OP_IOTA_COL) {
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int i = 0; i < V; ++i) acc[u][i] = u2f(ck.col0[u] + i);
        } else if constexpr (op == OP_IOTA_ROW) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t r = (ck.row[u] / scal(imm)) % scal(imm + 1);
#pragma unroll
                for (int i = 0; i < V; ++i) acc[u][i] = u2f(r);
            }
        } else if constexpr (op == OP_PHILOX) {
            // Philox4x32-10 (Salmon et al., SC'11).  A chunk starts on a multiple of eight elements, so it
            // takes the four words of counter blocks flat0/4 and flat0/4 + 1.  All 2U blocks of the thread
            // advance round by round together: they share the key schedule and give the scheduler 2U
            // independent multiply chains.
            uint32_t c[2 * U][4];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint64_t q = ck.flat0[u] >> 2;
                c[2 * u][0] = (uint32_t)q; c[2 * u][1] = (uint32_t)(q >> 32);
                c[2 * u + 1][0] = (uint32_t)(q + 1); c[2 * u + 1][1] = (uint32_t)((q + 1) >> 32);
                c[2 * u][2] = c[2 * u + 1][2] = scal(imm + 2);
                c[2 * u][3] = c[2 * u + 1][3] = scal(imm + 3);
            }
            uint32_t k0 = scal(imm), k1 = scal(imm + 1);
#pragma unroll
            for (int r = 0; r < 10; ++r) {
#pragma unroll
                for (int b = 0; b < 2 * U; ++b) {
                    const uint32_t hi0 = __umulhi(0xD2511F53u, c[b][0]), lo0 = 0xD2511F53u * c[b][0];
                    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c[b][2]), lo1 = 0xCD9E8D57u * c[b][2];
                    c[b][0] = hi1 ^ c[b][1] ^ k0;
                    c[b][1] = lo1;
                    c[b][2] = hi0 ^ c[b][3] ^ k1;
                    c[b][3] = lo0;
                }
                k0 += 0x9E3779B9u;
                k1 += 0xBB67AE85u;
            }
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    acc[u][i] = u2f(c[2 * u][i]);
                    acc[u][4 + i] = u2f(c[2 * u + 1][i]);
                }
        } else if constexpr (op >= OP_RED_SUM && op <= OP_RED_MIN) {
            red.template operator()<op - OP_RED_SUM, U, GUARD>(acc, ck.ok);
        } else if constexpr (op == OP_U_SQUARE) {
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int i = 0; i < V; i += 2) f2c_pair<F2_MUL, FLAV>(acc[u][i], acc[u][i + 1], acc[u][i], acc[u][i + 1]);
        } else if constexpr (op >= OP_U_NEG && op <= OP_C_NZI) {
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int i = 0; i < V; ++i) acc[u][i] = unc<op, FLAV>(acc[u][i]);
        } else if constexpr (I::is_ld(op)) {
            constexpr int d = op - OP_LD;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if constexpr (d < NT) operand_of<K>(t[d][u], u);
                else operand_of<K>(acc[u], u);
            }
        } else if constexpr (I::is_f2m(op)) {
            constexpr int k = op - OP_F2M;
            constexpr int f = k == F2M_ADD ? F2_ADD : k == F2M_SUB ? F2_SUB : k == F2M_RSUB ? F2_RSUB : F2_MUL;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float m[V];
                operand_of<K>(m, u);
#pragma unroll
                for (int i = 0; i < V; i += 2) f2c_pair<f, FLAV>(acc[u][i], acc[u][i + 1], m[i], m[i + 1]);
            }
        } else if constexpr (op >= OP_F2 && op < OP_I2) {
            constexpr int idx = (op - OP_F2) / LT_VM_NSRC, src = (op - OP_F2) % LT_VM_NSRC;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float m[V];
                source<src, imm>(m, u);
#pragma unroll
                for (int i = 0; i < V; i += 2) f2c_pair<idx, FLAV>(acc[u][i], acc[u][i + 1], m[i], m[i + 1]);
            }
        } else if constexpr (op >= OP_I2 && op < OP_CMP) {
            constexpr int idx = (op - OP_I2) / LT_VM_NSRC, src = (op - OP_I2) % LT_VM_NSRC;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float m[V];
                source<src, imm>(m, u);
#pragma unroll
                for (int i = 0; i < V; ++i) acc[u][i] = i2<idx>(acc[u][i], m[i]);
            }
        } else if constexpr (op >= OP_CMP && op < OP_WHERE_A) {
            constexpr int idx = (op - OP_CMP) / LT_VM_NSRC, src = (op - OP_CMP) % LT_VM_NSRC;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float m[V];
                source<src, imm>(m, u);
#pragma unroll
                for (int i = 0; i < V; ++i) acc[u][i] = cmp<idx>(acc[u][i], m[i]);
            }
        } else if constexpr (op >= OP_WHERE_A && op < OP_LIMIT) {
            constexpr bool variant_b = op >= OP_WHERE_B;
            constexpr int rel = variant_b ? op - OP_WHERE_B : op - OP_WHERE_A;
            constexpr int mt = rel / LT_VM_NSRC, src = rel % LT_VM_NSRC;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float m[V], msk[V];
                source<src, imm>(m, u);
                source<mt, 0>(msk, u);
#pragma unroll
                for (int i = 0; i < V; ++i) {
                    const bool on = f2u(msk[i]) != 0u;
                    acc[u][i] = variant_b ? (on ? m[i] : acc[u][i]) : (on ? acc[u][i] : m[i]);
                }
            }
        } else {
            static_assert(op == OP_END, "opcode not handled by the compiled shells");
        }
    }

    template <int K = PG::n_pro>
    __device__ __forceinline__ void run() {
        if constexpr (K < PG::n_ins) {
            step<K>();
            run<K + 1>();
        }
    }

    // Long rows (see lt_c_longrow): the program is run once per reduction plus once more.  In pass PHASE every
    // reduction before the PHASE-th yields its known result (red.val), the PHASE-th folds this thread's lanes into
    // red.part and ends the pass, and stores happen only in the last pass (the compiler drops whatever a pass
    // computes without using it).
    template <int PHASE, int K = PG::n_pro>
    __device__ __forceinline__ void run_phase() {
        if constexpr (K < PG::n_ins) {
            constexpr uint32_t op = PG::ins[K].op;
            if constexpr (I::is_red(op)) {
                constexpr int ord = I::red_ordinal(K);
                if constexpr (ord < PHASE) {
#pragma unroll
                    for (int u = 0; u < U; ++u)
#pragma unroll
                        for (int i = 0; i < V; ++i) acc[u][i] = red.val[ord];
                    run_phase<PHASE, K + 1>();
                } else {
                    constexpr int KIND = op - OP_RED_SUM;
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const float l0 = GroupReduce::red_comb<KIND>(acc[u][0], acc[u][1]), l1 = GroupReduce::red_comb<KIND>(acc[u][2], acc[u][3]);
                        const float l2 = GroupReduce::red_comb<KIND>(acc[u][4], acc[u][5]), l3 = GroupReduce::red_comb<KIND>(acc[u][6], acc[u][7]);
                        const float c = GroupReduce::red_comb<KIND>(GroupReduce::red_comb<KIND>(l0, l1), GroupReduce::red_comb<KIND>(l2, l3));
                        if (!GUARD || ck.ok[u]) red.part = GroupReduce::red_comb<KIND>(red.part, c);
                    }
                }
            } else if constexpr (op == OP_ST && PHASE < I::n_reds()) {
                run_phase<PHASE, K + 1>();
            } else {
                step<K>();
                run_phase<PHASE, K + 1>();
            }
        }
    }

    // storage-format chunks of the full-class inputs from a row staged in shared memory; soff[s] is the byte
    // offset of slot s's row inside the stage
    template <int K = PG::n_pro>
    __device__ __forceinline__ void fetch_row(const unsigned char *stage, const uint32_t (&soff)[PG::n_slots]) {
        if constexpr (K < PG::n_ins) {
            constexpr uint32_t op = PG::ins[K].op;
            if constexpr (I::is_ld(op) || I::is_f2m(op)) {
                constexpr int slot = PG::ins[K].imm;
                if constexpr (PG::cls[slot] == LT_CLS_FULL) {
                    constexpr int cb = I::chunk_bytes(slot), sh = esz_shift(PG::dtype[slot]);
                    constexpr int ord = I::load_ordinal(K);
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        if (GUARD && !ck.ok[u]) continue;
                        const unsigned char *b = stage + soff[slot] + ((size_t)ck.col0[u] << sh);
                        if constexpr (cb == 8) {
                            const uint2 w = *reinterpret_cast<const uint2 *>(b);
                            raw[ord][u].a.x = w.x;
                            raw[ord][u].a.y = w.y;
                        } else {
                            raw[ord][u].a = *reinterpret_cast<const uint4 *>(b);
                            if constexpr (cb == 32) raw[ord][u].b = *reinterpret_cast<const uint4 *>(b + 16);
                        }
                    }
                }
            }
            fetch_row<K + 1>(stage, soff);
        }
    }
};

// State of the reductions of a long row: results so far, and this thread's share of the one being formed.
struct LongRed {
    float val[4];
    float part;
};

struct ScalK {
    const LtKParams &P;
    __device__ __forceinline__ uint32_t operator()(uint32_t i) const { return P.scal[i]; }
};
struct PtrK {
    const LtKParams &P;
    __device__ __forceinline__ uint64_t operator()(uint32_t s) const { return P.ptr[s]; }
    __device__ __forceinline__ uint32_t pitch(uint32_t s) const { return P.pitch[s]; }
    // elements a slot of the class holds (bounds checks of the debug build)
    __device__ __forceinline__ uint64_t extent(int cls) const {
        return cls == LT_CLS_FULL ? P.n : cls == LT_CLS_COLVEC ? P.cols : cls == LT_CLS_ROWVEC ? P.rows : 1;
    }
};
struct ScalM {
    const LtMultiParams &P;
    __device__ __forceinline__ uint32_t operator()(uint32_t i) const { return P.scal[i]; }
};
struct PtrM {
    const LtMultiParams &P;
    uint32_t base;
    uint32_t numel;
    __device__ __forceinline__ uint64_t operator()(uint32_t s) const { return P.ptr[base + s]; }
    __device__ __forceinline__ uint32_t pitch(uint32_t) const { return 0; }
    __device__ __forceinline__ uint64_t extent(int) const { return numel; }
};

template <class PG, int U, int T = 0, class M>
__device__ __forceinline__ void hoist_colvecs(const M &m, float (&hv)[NT][U][V]) {
    if constexpr (T < NT) {
        if constexpr (Info<PG>::pro_slot(T) >= 0) {
#pragma unroll
            for (int u = 0; u < U; ++u) m.template load_now<Info<PG>::pro_slot(T)>(hv[T][u], u);
        }
        hoist_colvecs<PG, U, T + 1>(m, hv);
    }
}

template <class PG, int U, int T = 0, class M>
__device__ __forceinline__ void hoist_to_shared(const M &m, float *base) {
    if constexpr (T < NT) {
        if constexpr (Info<PG>::pro_slot(T) >= 0) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float d[V];
                m.template load_now<Info<PG>::pro_slot(T)>(d, u);
                float4 *q = reinterpret_cast<float4 *>(base + ((Info<PG>::reserved_ordinal(T) * U + u) * C_ROW_THREADS + threadIdx.x) * V);
                q[0] = make_float4(d[0], d[1], d[2], d[3]);
                q[1] = make_float4(d[4], d[5], d[6], d[7]);
            }
        }
        hoist_to_shared<PG, U, T + 1>(m, base);
    }
}

struct TrueTag { static constexpr bool value = true; };
struct FalseTag { static constexpr bool value = false; };

// ------------------------------------------------------------------ shells
// Elementwise: chunk c of U-tuples strides through the tensor; rows are a multiple of the chunk.
template <class PG, int U>
__global__ void __launch_bounds__(C_THREADS) lt_c_ew(const __grid_constant__ LtKParams P) {
    const uint32_t n_chunks = (uint32_t)P.n_chunks;
    const uint32_t stride = gridDim.x * C_THREADS;
    const PtrK ptr{P};
    const ScalK scal{P};
    NoReduce red;
    pdl_release();
    pdl_wait();
    for (uint32_t c = blockIdx.x * C_THREADS + threadIdx.x; c < n_chunks; c += U * stride) {
        Coords<U> ck;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t cx = c + u * stride;
            ck.ok[u] = cx < n_chunks;
            const uint32_t cu = ck.ok[u] ? cx : 0u;  // a chunk past the end takes the coordinates of chunk 0 (see lt_c_row)
            ck.flat0[u] = (uint64_t)cu * V;
            if (Info<PG>::needs_coords() && P.rowcol) {
                const uint32_t q = __umulhi(P.div_mul, cu);
                const uint32_t row = (q + ((cu - q) >> P.div_sh1)) >> P.div_sh2;
                ck.row[u] = row;
                ck.col0[u] = (cu - row * P.cpr) * V;
            } else {
                ck.row[u] = 0;
                ck.col0[u] = cu * V;
            }
        }
        Machine<PG, U, PtrK, ScalK, NoReduce> m(ptr, scal, red, ck);
        m.issue_loads();
        m.run();
    }
}

// Row reductions: thread `gl` of a row's group owns chunks gl, gl + group, ... of the row.
// With `depth` > 0 the full-class inputs of the CTA's next `depth` blocks of rows are in flight as
// asynchronous copies into a ring of shared-memory stages while the current block is computed.
// (programs with column vectors at up to four chunks per thread: capped at 128 registers, four CTAs per SM instead of three --
// LayerNorm bf16 at 2048 columns 102 -> 92 us; 0 = no hint, the others measured slower or equal with one)
template <class PG, int U>
__global__ void __launch_bounds__(C_ROW_THREADS, (U <= 4 && Info<PG>::n_reserved() > 0) ? 4 : 0) lt_c_row(const __grid_constant__ LtKParams P, uint32_t group, uint32_t group_log2,
                                                          uint32_t depth) {
    __shared__ float red_buf[64];
    extern __shared__ __align__(16) unsigned char stage_mem[];
    using M = Machine<PG, U, PtrK, ScalK, GroupReduce>;
    constexpr uint32_t STAGE = Info<PG>::stage_bytes(U, C_ROW_THREADS);
    const PtrK ptr{P};
    const ScalK scal{P};
    GroupReduce red{red_buf, group, 0u};
    const uint32_t rows_per_cta = blockDim.x >> group_log2;
    const uint32_t row_blocks = (P.rows + rows_per_cta - 1u) / rows_per_cta;
    const uint32_t sub = threadIdx.x >> group_log2, gl = threadIdx.x & (group - 1u);
    auto coords_of = [&](uint32_t rb, Coords<U> &ck) {
        const uint32_t row = rb * rows_per_cta + sub;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            // a chunk past the end of the row, or a row past the last, takes the coordinates of an existing
            // one: broadcast operands are read at use without a validity test and must stay in bounds
            const uint32_t col = (u * group + gl) * V;
            const bool in_row = col < P.cols, in_rows = row < P.rows;
            ck.row[u] = in_rows ? row : 0u;
            ck.col0[u] = in_row ? col : 0u;
            ck.ok[u] = in_rows && in_row;
            ck.flat0[u] = (uint64_t)ck.row[u] * P.cols + ck.col0[u];
        }
    };
    const uint32_t stage0 = (uint32_t)__cvta_generic_to_shared(stage_mem);
    pdl_release();
    pdl_wait();
    if (depth) {  // requires blockDim.x == C_ROW_THREADS
        uint32_t rb = blockIdx.x;
        for (uint32_t d = 0; d < depth; ++d, rb += gridDim.x) {
            if (rb < row_blocks) {
                Coords<U> nx;
                coords_of(rb, nx);
                M::template stage_issue<C_ROW_THREADS>(ptr, nx.flat0, nx.ok, stage0 + d * STAGE);
            }
            cp_async_commit();
        }
    }
    // every thread owns U whole chunks of an existing row in every iteration: no validity tests
    const bool full = (P.rows % rows_per_cta) == 0 && group * U * V == P.cols;
    uint32_t s = 0;
    // Column vectors of the reserved temporaries (gamma, beta, a bias): a thread owns the same columns in every
    // iteration, so when they fit in 64 registers they are loaded once instead of being re-read through L1 for every
    // row -- two f32 vectors are 8 bytes per element of L1 traffic, twice the HBM traffic of a bf16 LayerNorm.  Not
    // for programs that generate random bits: they are short of registers and issue slots, not of L1 bandwidth.
    constexpr bool HOIST = Info<PG>::n_reserved() > 0 && Info<PG>::n_reserved() * U * V <= 64 && !Info<PG>::integer_heavy();
    float hv[NT][U][V];
    if constexpr (HOIST) {
        Coords<U> c0;
        coords_of(0, c0);
        Machine<PG, U, PtrK, ScalK, GroupReduce, true> m0(ptr, scal, red, c0);
        hoist_colvecs<PG, U>(m0, hv);
    }
    auto iterate = [&](auto guard_tag) {
        constexpr bool GUARD = decltype(guard_tag)::value;
        using MG = Machine<PG, U, PtrK, ScalK, GroupReduce, GUARD, HOIST ? 1 : 0>;
        for (uint32_t rb = blockIdx.x; rb < row_blocks; rb += gridDim.x) {
            Coords<U> ck;
            coords_of(rb, ck);
            MG m(ptr, scal, red, ck);
            m.hoisted = hv;
            if (depth) {
                cp_async_wait(depth - 1);
                m.template stage_fetch<C_ROW_THREADS>(stage_mem + s * STAGE);
                // the stage just read is refilled with the block `depth` iterations ahead
                const uint32_t rn = rb + depth * gridDim.x;
                if (rn < row_blocks) {
                    Coords<U> nx;
                    coords_of(rn, nx);
                    MG::template stage_issue<C_ROW_THREADS>(ptr, nx.flat0, nx.ok, stage0 + s * STAGE);
                }
                cp_async_commit();
                s = s + 1 == depth ? 0 : s + 1;
            } else {
                m.issue_loads();
            }
            m.run();
        }
    };
    if (full) iterate(FalseTag{});
    else iterate(TrueTag{});
    if (depth) cp_async_wait(0);
}

// An elementwise program whose result is reduced over the rows of every column, or over everything, instead of
// being stored (LT_CLS_REDUCED): the first of two stages.  Columns: CTA (bx, by) of 32 x 8 threads takes the 32 chunks
// of columns bx * 256 .. and the rows [by * rows_per, ..); thread (x, y) owns one chunk of eight columns and walks rows
// y, y + 8, .., two at a time; the eight row lanes meet in shared memory and the CTA writes one binary64 partial per
// column to partial[by * cols + col].  Everything: chunks strided over the grid, partial[bx] per CTA.  The partials
// are what lt_reduce_cols / lt_reduce_all of reduce.cu read in their second stage.  Rows are whole chunks.
// writes the partial results of the ORD-th reduced value (see lt_c_ewred), then those of the next
template <class PG, int ORD, class R>
__device__ __forceinline__ void ewred_finish(const LtKParams &P, const R &red, double *smem) {
    if constexpr (ORD < Info<PG>::n_accum()) {
        constexpr int SLOT = Info<PG>::accum_slot_at(ORD), KIND = Info<PG>::accum_kind_of(SLOT);
        using Ops = AccumOps<KIND>;
        double *partial = reinterpret_cast<double *>(P.ptr[SLOT]);
        if constexpr (ORD > 0) __syncthreads();  // the previous value's partials have been read
        if constexpr (Info<PG>::accum_axis() == 0) {
            const uint32_t x = threadIdx.x & 31u, y = threadIdx.x >> 5;
#pragma unroll
            for (int i = 0; i < V; ++i) smem[y * (32 * V + 1) + x * V + i] = red.template get<ORD, KIND>(i);
            __syncthreads();
            const uint32_t col = blockIdx.x * 32u * V + threadIdx.x;  // 256 threads, 256 columns
            if (col < P.cols) {
                double v = smem[threadIdx.x];
#pragma unroll
                for (int k = 1; k < 8; ++k) v = Ops::comb(v, smem[k * (32 * V + 1) + threadIdx.x]);
                partial[(uint64_t)blockIdx.y * P.cols + col] = v;
            }
        } else {
            double v = Ops::comb(Ops::comb(Ops::comb(red.template get<ORD, KIND>(0), red.template get<ORD, KIND>(1)),
                                           Ops::comb(red.template get<ORD, KIND>(2), red.template get<ORD, KIND>(3))),
                                 Ops::comb(Ops::comb(red.template get<ORD, KIND>(4), red.template get<ORD, KIND>(5)),
                                           Ops::comb(red.template get<ORD, KIND>(6), red.template get<ORD, KIND>(7))));
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) v = Ops::comb(v, __shfl_xor_sync(0xffffffffu, v, off));
            if ((threadIdx.x & 31u) == 0) smem[threadIdx.x >> 5] = v;
            __syncthreads();
            if (threadIdx.x == 0) {
                double r = smem[0];
                for (int w = 1; w < C_THREADS / 32; ++w) r = Ops::comb(r, smem[w]);
                partial[blockIdx.x] = r;
            }
        }
        ewred_finish<PG, ORD + 1>(P, red, smem);
    }
}

template <class PG, int ORD, class R>
__device__ __forceinline__ void ewred_reset(R &red) {
    if constexpr (ORD < Info<PG>::n_accum()) {
        red.template reset<ORD, Info<PG>::accum_kind_of(Info<PG>::accum_slot_at(ORD))>();
        ewred_reset<PG, ORD + 1>(red);
    }
}

template <class PG>
__global__ void __launch_bounds__(C_THREADS) lt_c_ewred(const __grid_constant__ LtKParams P, uint32_t rows_per) {
    constexpr int AXIS = Info<PG>::accum_axis();
    static_assert(Info<PG>::n_accum() >= 1 && Info<PG>::n_accum() <= C_MAX_REDUCED, "reduced values per program");
    using R = AccumSet<Info<PG>::n_accum()>;
    __shared__ double smem[AXIS == 0 ? 8 * (32 * V + 1) : C_THREADS / 32];
    const PtrK ptr{P};
    const ScalK scal{P};
    R red;
    ewred_reset<PG, 0>(red);
    pdl_release();
    pdl_wait();
    if constexpr (AXIS == 0) {
        const uint32_t x = threadIdx.x & 31u, y = threadIdx.x >> 5;
        const uint32_t cchunk = blockIdx.x * 32u + x;
        const uint32_t r0 = blockIdx.y * rows_per;
        const uint32_t r1 = r0 + rows_per < P.rows ? r0 + rows_per : P.rows;
        if (cchunk < P.cpr) {
            for (uint32_t r = r0 + y; r < r1; r += 16) {
                Coords<2> ck;
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const uint32_t row = r + 8u * u;
                    ck.ok[u] = row < r1;
                    ck.row[u] = ck.ok[u] ? row : r;
                    ck.col0[u] = cchunk * V;
                    ck.flat0[u] = (uint64_t)ck.row[u] * P.cols + ck.col0[u];
                }
                Machine<PG, 2, PtrK, ScalK, R, true> m(ptr, scal, red, ck);
                m.issue_loads();
                m.run();
            }
        }
    } else {
        const uint32_t n_chunks = (uint32_t)P.n_chunks;
        const uint32_t stride = gridDim.x * C_THREADS;
        for (uint32_t c = blockIdx.x * C_THREADS + threadIdx.x; c < n_chunks; c += 2 * stride) {
            Coords<2> ck;
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const uint32_t cx = c + u * stride;
                ck.ok[u] = cx < n_chunks;
                const uint32_t cu = ck.ok[u] ? cx : 0u;
                ck.flat0[u] = (uint64_t)cu * V;
                if (Info<PG>::needs_coords() && P.rowcol) {
                    const uint32_t q = __umulhi(P.div_mul, cu);
                    const uint32_t row = (q + ((cu - q) >> P.div_sh1)) >> P.div_sh2;
                    ck.row[u] = row;
                    ck.col0[u] = (cu - row * P.cpr) * V;
                } else {
                    ck.row[u] = 0;
                    ck.col0[u] = cu * V;
                }
            }
            Machine<PG, 2, PtrK, ScalK, R, true> m(ptr, scal, red, ck);
            m.issue_loads();
            m.run();
        }
    }
    ewred_finish<PG, 0>(P, red, smem);
}

// Multi-tensor: every tensor is a flat range of chunks; a super-chunk is 2048 consecutive chunks.
template <class PG, int U>
__global__ void __launch_bounds__(C_THREADS) lt_c_multi(const __grid_constant__ LtMultiParams P) {
    const ScalM scal{P};
    NoReduce red;
    constexpr uint32_t PER_SUPER = LT_EW_THREADS * LT_MULTI_SUB;
    static_assert(LT_EW_THREADS == C_THREADS && LT_MULTI_SUB % U == 0, "super-chunk walk");
    pdl_release();
    pdl_wait();
    for (uint32_t sc = blockIdx.x; sc < P.total_super; sc += gridDim.x) {
        uint32_t lo = 0, hi = P.n_inst;
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (P.super_prefix[mid] <= sc) lo = mid; else hi = mid;
        }
        const PtrM ptr{P, lo * P.n_slots, P.numel[lo]};
        const uint32_t chunks_all = P.numel[lo] / V;
        const uint32_t first = (sc - P.super_prefix[lo]) * PER_SUPER + threadIdx.x;
#pragma unroll 1
        for (uint32_t k = 0; k < LT_MULTI_SUB; k += U) {
            Coords<U> ck;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t cu = first + (k + u) * C_THREADS;
                ck.ok[u] = cu < chunks_all;
                ck.flat0[u] = (uint64_t)cu * V;
                ck.row[u] = 0;
                ck.col0[u] = cu * V;
            }
            if (!ck.ok[0]) break;
            Machine<PG, U, PtrM, ScalM, NoReduce> m(ptr, scal, red, ck);
            m.issue_loads();
            m.run();
        }
    }
}


// ------------------------------------------------------------------ long rows
// A word the host reads after a blocking call: bit 0 = a bounded wait for an asynchronous copy gave up.
__device__ unsigned int lt_device_status = 0;

__device__ __forceinline__ uint64_t global_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Waits until the phase of the mbarrier at shared address `bar` with parity `parity` has completed, for at most
// `limit_ns` nanoseconds.  Returns false when it gave up.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint64_t limit_ns) {
    const uint64_t t0 = global_ns();
    for (;;) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (done) return true;
        if (global_ns() - t0 > limit_ns) return false;
    }
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// One-dimensional bulk asynchronous copy global -> this CTA's shared memory (no multicast); both addresses and the
// size are multiples of 16 bytes.  Completion is counted in bytes on the mbarrier.
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst), "l"(src),
                 "r"(bytes), "r"(bar)
                 : "memory");
}

constexpr int C_LONG_U = 2;  // chunks per thread and slice; CTAs of 256 threads, or 512 when only one fits an SM
constexpr uint32_t C_LONG_MAX_BULK = 1u << 19;  // keeps a stage's byte count inside the mbarrier's transaction counter

// compile-time walks over the slots of a program (the program tables are not addressable at run time in device code)
template <class PG, int S = 0>
__device__ __forceinline__ void long_offsets(uint32_t cols, uint32_t (&soff)[PG::n_slots], uint32_t off) {
    if constexpr (S < PG::n_slots) {
        soff[S] = off;
        if constexpr (Info<PG>::full_input(S)) off += (cols * Info<PG>::elem_bytes(S) + 15u) & ~15u;
        long_offsets<PG, S + 1>(cols, soff, off);
    }
}
template <class PG, int S = 0>
__device__ __forceinline__ uint32_t long_row_bytes(uint32_t cols) {
    if constexpr (S < PG::n_slots) {
        uint32_t here = 0;
        if constexpr (Info<PG>::full_input(S)) here = cols * Info<PG>::elem_bytes(S);
        return here + long_row_bytes<PG, S + 1>(cols);
    } else {
        return 0u;
    }
}
template <class PG, int S = 0, class Ptr>
__device__ __forceinline__ void long_issue(const Ptr &ptr, uint32_t cols, uint32_t row, uint32_t stage, const uint32_t (&soff)[PG::n_slots],
                                           uint32_t bar) {
    if constexpr (S < PG::n_slots) {
        if constexpr (Info<PG>::full_input(S)) {
            const uint32_t bytes = cols * Info<PG>::elem_bytes(S);
            const char *src = reinterpret_cast<const char *>(ptr(S)) + (uint64_t)row * bytes;
            for (uint32_t done = 0; done < bytes; done += C_LONG_MAX_BULK) {
                const uint32_t n = bytes - done < C_LONG_MAX_BULK ? bytes - done : C_LONG_MAX_BULK;
                bulk_copy_g2s(stage + soff[S] + done, src + done, n, bar);
            }
        }
        long_issue<PG, S + 1>(ptr, cols, row, stage, soff, bar);
    }
}

// Asks for `bytes` (a multiple of 16) at `src` to be brought into L2; nothing waits for it.
__device__ __forceinline__ void bulk_prefetch_l2(const void *src, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}
template <class PG, int S = 0, class Ptr>
__device__ __forceinline__ void long_prefetch(const Ptr &ptr, uint32_t cols, uint32_t row) {
    if constexpr (S < PG::n_slots) {
        if constexpr (Info<PG>::full_input(S)) {
            const uint32_t bytes = cols * Info<PG>::elem_bytes(S);
            const char *src = reinterpret_cast<const char *>(ptr(S)) + (uint64_t)row * bytes;
            for (uint32_t done = 0; done < bytes; done += C_LONG_MAX_BULK)
                bulk_prefetch_l2(src + done, bytes - done < C_LONG_MAX_BULK ? bytes - done : C_LONG_MAX_BULK);
        }
        long_prefetch<PG, S + 1>(ptr, cols, row);
    }
}

template <int KIND, int T>
__device__ __forceinline__ float long_cta_reduce(float v, float *buf) {
#pragma unroll
    for (uint32_t off = 16; off > 0; off >>= 1) v = GroupReduce::red_comb<KIND>(v, __shfl_xor_sync(0xffffffffu, v, off));
    __syncthreads();  // buf may still be read from the previous reduction
    if ((threadIdx.x & 31u) == 0) buf[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = buf[0];
#pragma unroll
    for (int w = 1; w < T / 32; ++w) r = GroupReduce::red_comb<KIND>(r, buf[w]);
    return r;
}

// Rows too long for a thread group's registers: a CTA of T threads owns a row and walks it in slices of T x 2 chunks.  A program
// with n reductions makes n + 1 passes over the row (Machine::run_phase).  With `depth` > 0 the row's full-class
// inputs are brought into shared memory once, by one-dimensional bulk asynchronous copies that complete on an
// mbarrier, `depth` rows ahead; every pass then reads the staged row.  With depth 0 the passes read global memory
// (the row was just read by this CTA and sits in L2).  The wait for a stage is bounded: when it gives up the CTA
// raises bit 0 of lt_device_status, waits (again bounded) for the copies it still has in flight and returns.
// `l2_ahead` (when the rows are multiples of 16 bytes): while a row is processed, the row the CTA stages or reads
// next is requested into L2, so that HBM keeps streaming during the passes that read no global memory.
template <class PG, int T>
__global__ void __launch_bounds__(T) lt_c_longrow(const __grid_constant__ LtKParams P, uint32_t depth, uint32_t stage_bytes,
                                                  uint64_t limit_ns, uint32_t l2_ahead) {
    constexpr int U = C_LONG_U, NR = Info<PG>::n_reds();
    static_assert(NR <= 4, "at most four reductions per long-row program");
    using M = Machine<PG, U, PtrK, ScalK, LongRed, true>;
    __shared__ float red_buf[T / 32];
    __shared__ __align__(8) uint64_t bars[2];
    extern __shared__ __align__(128) unsigned char stage_mem[];
    const PtrK ptr{P};
    const ScalK scal{P};
    LongRed red;
    const uint32_t cpr = P.cpr, n_slices = (cpr + T * U - 1) / (T * U);
    // byte offset of every staged slot's row inside a stage
    uint32_t soff[PG::n_slots];
    long_offsets<PG>(P.cols, soff, 0u);
    const uint32_t bar0 = (uint32_t)__cvta_generic_to_shared(&bars[0]);
    const uint32_t stage0 = (uint32_t)__cvta_generic_to_shared(stage_mem);
    if (depth && threadIdx.x == 0) {
        mbar_init(bar0, 1);
        mbar_init(bar0 + 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    pdl_release();
    pdl_wait();
    __syncthreads();
    auto issue = [&](uint32_t row, uint32_t s) {  // thread 0: start the copies of `row` into stage s
        mbar_expect_tx(bar0 + 8 * s, long_row_bytes<PG>(P.cols));
        long_issue<PG>(ptr, P.cols, row, stage0 + s * stage_bytes, soff, bar0 + 8 * s);
    };
    if (depth && threadIdx.x == 0) {
        uint32_t row = blockIdx.x;
        for (uint32_t d = 0; d < depth; ++d, row += gridDim.x)
            if (row < P.rows) issue(row, d);
    }
    uint32_t k = 0;
    for (uint32_t row = blockIdx.x; row < P.rows; row += gridDim.x, ++k) {
        const uint32_t s = depth ? k % depth : 0u;
        const unsigned char *stage = stage_mem + (size_t)s * stage_bytes;
        if (l2_ahead && threadIdx.x == 0) {
            const uint32_t ahead = row + (depth ? depth : 1u) * gridDim.x;  // not yet requested by a copy into shared memory
            if (ahead < P.rows) long_prefetch<PG>(ptr, P.cols, ahead);
        }
        if (depth) {
            const bool landed = mbar_wait_bounded(bar0 + 8 * s, (k / depth) & 1u, limit_ns);
            if (__syncthreads_or(landed ? 0 : 1)) {
                if (threadIdx.x == 0) atomicOr(&lt_device_status, 1u);
                // copies this CTA still has in flight write into its shared memory: give them the same time once more
                for (uint32_t d = 0; d < depth; ++d) mbar_wait_bounded(bar0 + 8 * d, ((k + (d >= s ? 0u : 1u)) / depth) & 1u, limit_ns);
                return;
            }
        }
        auto pass = [&](auto phase_tag) {
            constexpr int PHASE = decltype(phase_tag)::value;
            if constexpr (PHASE < NR) red.part = Info<PG>::red_kind(PHASE) == 0 ? 0.0f : (Info<PG>::red_kind(PHASE) == 1 ? -LT_INF : LT_INF);
            for (uint32_t sl = 0; sl < n_slices; ++sl) {
                Coords<U> ck;
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const uint32_t chunk = (sl * U + u) * T + threadIdx.x;
                    ck.ok[u] = chunk < cpr;
                    ck.row[u] = row;
                    ck.col0[u] = ck.ok[u] ? chunk * V : 0u;  // a chunk past the end takes the coordinates of the first
                    ck.flat0[u] = (uint64_t)row * P.cols + ck.col0[u];
                }
                M m(ptr, scal, red, ck);
                if (depth) m.fetch_row(stage, soff);
                else m.issue_loads();
                m.template run_phase<PHASE>();
            }
            if constexpr (PHASE < NR) red.val[PHASE] = long_cta_reduce<Info<PG>::red_kind(PHASE), T>(red.part, red_buf);
        };
        pass(IntTag<0>{});
        if constexpr (NR >= 1) pass(IntTag<1>{});
        if constexpr (NR >= 2) pass(IntTag<2>{});
        if constexpr (NR >= 3) pass(IntTag<3>{});
        if constexpr (NR >= 4) pass(IntTag<4>{});
        if (depth) {
            __syncthreads();  // every thread has finished reading stage s
            const uint32_t next = row + depth * gridDim.x;
            if (threadIdx.x == 0 && next < P.rows) issue(next, s);
        }
    }
}

// ------------------------------------------------------------------ long rows in the registers of a thread-block cluster
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_id_x() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_count_x() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(r));
    return r;
}
// The cluster's hardware barrier (all threads of all its CTAs arrive; like bar.sync it completes by itself under
// uniform control flow).  Used at the two ends of the kernel only: its release semantics wait for every earlier
// global store of the thread, far too expensive per row.
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// A 32-bit store into the shared memory of CTA `cta_rank` of the cluster (distributed shared memory) that, when it
// lands, counts four bytes on an mbarrier of that CTA: whoever sees the barrier's phase complete sees the value.
// `slot` and `bar` are this CTA's shared-window addresses of the word and the barrier; the peer's are at the same
// offsets.  No fence is involved, so earlier global stores of the thread stay in flight.
__device__ __forceinline__ void store_remote_signal(uint32_t slot, uint32_t bar, uint32_t cta_rank, float v) {
    uint32_t rs, rb;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rs) : "r"(slot), "r"(cta_rank));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rb) : "r"(bar), "r"(cta_rank));
    asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.f32 [%0], %1, [%2];" ::"r"(rs), "f"(v), "r"(rb) : "memory");
}

constexpr int C_MAX_CLUSTER = 8;                     // portable cluster size
constexpr int C_ROW_WARPS = C_ROW_THREADS / 32;

// Row reductions of a thread group that spans all threads of all CTAs of a cluster.  Lanes, chunks and the warp are
// folded as in GroupReduce.  Then lane k of every warp sends the warp's partial to CTA k of the cluster, into slot
// [sender's rank][warp] of one of two exchange buffers, as a store that signals an mbarrier there; a thread waits
// (bounded) until its CTA's barrier has counted the bytes of all warps of all CTAs and folds the slots in index
// order -- the same order everywhere, so every thread of the row holds the same bits.  No CTA-wide or cluster-wide
// barrier per reduction.  Buffers and barriers alternate between consecutive reductions; a buffer is written again
// two reductions later, and a CTA sends for reduction n + 2 only after it has received every CTA's part of n + 1,
// which each sent after all its threads had finished reading n.
struct ClusterReduce {
    const float *slots;   // 2 x (C_MAX_CLUSTER x C_ROW_WARPS) floats
    uint32_t slots_addr;  // shared-window address of `slots`
    uint32_t bar_addr;    // ... of the two mbarriers
    uint32_t nctas, rank, phase;
    uint64_t limit_ns;
    bool gave_up;
    template <int KIND, int U, bool GUARD>
    __device__ __forceinline__ void operator()(float (&acc)[U][V], const bool (&ok)[U]) {
        const float ident = KIND == 0 ? 0.0f : (KIND == 1 ? -LT_INF : LT_INF);
        float part[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            float l0 = GroupReduce::red_comb<KIND>(acc[u][0], acc[u][1]), l1 = GroupReduce::red_comb<KIND>(acc[u][2], acc[u][3]);
            float l2 = GroupReduce::red_comb<KIND>(acc[u][4], acc[u][5]), l3 = GroupReduce::red_comb<KIND>(acc[u][6], acc[u][7]);
            part[u] = (!GUARD || ok[u]) ? GroupReduce::red_comb<KIND>(GroupReduce::red_comb<KIND>(l0, l1), GroupReduce::red_comb<KIND>(l2, l3)) : ident;
        }
#pragma unroll
        for (int s = 1; s < U; s <<= 1)
#pragma unroll
            for (int u = 0; u + s < U; u += 2 * s) part[u] = GroupReduce::red_comb<KIND>(part[u], part[u + s]);
        float r = part[0];
#pragma unroll
        for (uint32_t off = 16; off > 0; off >>= 1) r = GroupReduce::red_comb<KIND>(r, __shfl_xor_sync(0xffffffffu, r, off));
        const uint32_t half = phase & 1u, parity = (phase >> 1) & 1u;
        ++phase;
        const uint32_t bar = bar_addr + 8u * half;
        const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
        if (threadIdx.x == 0) mbar_expect_tx(bar, nctas * C_ROW_WARPS * 4u);
        if (lane < nctas) store_remote_signal(slots_addr + ((half * C_MAX_CLUSTER + rank) * C_ROW_WARPS + warp) * 4u, bar, lane, r);
        if (!gave_up && !mbar_wait_bounded(bar, parity, limit_ns)) {
            gave_up = true;  // results from here on are wrong and the host is told; later waits are skipped
            atomicOr(&lt_device_status, 1u);
        }
        const float4 *x = reinterpret_cast<const float4 *>(slots + half * C_MAX_CLUSTER * C_ROW_WARPS);
        static_assert(C_ROW_WARPS == 4, "one 128-bit load per CTA's partials");
        float4 q = x[0];
        r = GroupReduce::red_comb<KIND>(GroupReduce::red_comb<KIND>(q.x, q.y), GroupReduce::red_comb<KIND>(q.z, q.w));
        for (uint32_t k = 1; k < nctas; ++k) {
            q = x[k];
            r = GroupReduce::red_comb<KIND>(r, GroupReduce::red_comb<KIND>(GroupReduce::red_comb<KIND>(q.x, q.y), GroupReduce::red_comb<KIND>(q.z, q.w)));
        }
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
            for (int i = 0; i < V; ++i) acc[u][i] = r;
    }
};

// Rows longer than one CTA's registers hold, up to 8 CTAs x 128 threads x 8 chunks x 8 elements = 65536 columns: the
// row's thread group is a thread-block cluster.  Thread t of CTA r (of K) owns chunks (u K + r) 128 + t, u = 0..U-1, of
// the row its cluster is working on and keeps them in registers across the reductions, exactly as in lt_c_row; only
// the reductions differ (ClusterReduce).  One pass over the data whatever the number of reductions; a thread owns
// the same columns for every row, so small column vectors are loaded once.  With `depth` > 0 the CTA's parts of the
// cluster's next `depth` rows are in flight as asynchronous copies into a ring of shared-memory stages.  All CTAs
// of a cluster run the same rows and the same program.  The kernel ends with the cluster's barrier: no CTA leaves
// while another may still write into its shared memory.
template <class PG, int U, bool HS>
__global__ void __launch_bounds__(C_ROW_THREADS, (U <= 4 && Info<PG>::n_reserved() > 0) ? 4 : 0) lt_c_rowc(const __grid_constant__ LtKParams P, uint32_t depth, uint64_t limit_ns) {
    __shared__ __align__(16) float slots[2 * C_MAX_CLUSTER * C_ROW_WARPS];
    __shared__ __align__(8) uint64_t bars[2];
    extern __shared__ __align__(16) unsigned char stage_mem[];
    constexpr uint32_t STAGE = Info<PG>::stage_bytes(U, C_ROW_THREADS);
    const PtrK ptr{P};
    const ScalK scal{P};
    const uint32_t nctas = cluster_nctarank(), rank = cluster_ctarank();
    const uint32_t group = nctas * C_ROW_THREADS, gl = rank * C_ROW_THREADS + threadIdx.x;
    const uint32_t first = cluster_id_x(), step = cluster_count_x();
    const uint32_t bar0 = (uint32_t)__cvta_generic_to_shared(bars);
    ClusterReduce red{slots, (uint32_t)__cvta_generic_to_shared(slots), bar0, nctas, rank, 0u, limit_ns, false};
    if (threadIdx.x == 0) {
        mbar_init(bar0, 1);
        mbar_init(bar0 + 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    auto coords_of = [&](uint32_t row, Coords<U> &ck) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t col = (u * group + gl) * V;
            const bool in_row = col < P.cols, in_rows = row < P.rows;  // a chunk that does not exist takes the coordinates of one that does
            ck.row[u] = in_rows ? row : 0u;
            ck.col0[u] = in_row ? col : 0u;
            ck.ok[u] = in_row && in_rows;
            ck.flat0[u] = (uint64_t)ck.row[u] * P.cols + ck.col0[u];
        }
    };
    // HS: the column vectors of the reserved temporaries (the thread's columns of gamma, beta, a bias) are kept in
    // shared memory, in front of the stages, instead of in registers: 32 bytes per vector and chunk for each thread
    constexpr uint32_t HOIST_BYTES = HS ? Info<PG>::n_reserved() * U * C_ROW_THREADS * V * 4 : 0;
    unsigned char *const ring = stage_mem + HOIST_BYTES;
    const uint32_t stage0 = (uint32_t)__cvta_generic_to_shared(ring);
    pdl_wait();
    cluster_sync();  // every CTA of the cluster is running, its barriers initialised, before one writes into another's shared memory
    using M = Machine<PG, U, PtrK, ScalK, ClusterReduce>;
    if (depth) {
        uint32_t row = first;
        for (uint32_t d = 0; d < depth; ++d, row += step) {
            if (row < P.rows) {
                Coords<U> nx;
                coords_of(row, nx);
                M::template stage_issue<C_ROW_THREADS>(ptr, nx.flat0, nx.ok, stage0 + d * STAGE);
            }
            cp_async_commit();
        }
    }
    const bool full = group * U * V == P.cols;
    constexpr int HOIST = Info<PG>::n_reserved() == 0 ? 0 : HS ? 2 : (Info<PG>::n_reserved() * U * V <= 64 && !Info<PG>::integer_heavy()) ? 1 : 0;
    float hv[NT][U][V];
    if constexpr (HOIST == 1) {
        Coords<U> c0;
        coords_of(0, c0);
        Machine<PG, U, PtrK, ScalK, ClusterReduce, true> m0(ptr, scal, red, c0);
        hoist_colvecs<PG, U>(m0, hv);
    } else if constexpr (HOIST == 2) {
        // every thread copies its own columns and later reads nothing else: no barrier needed
        Coords<U> c0;
        coords_of(0, c0);
        Machine<PG, U, PtrK, ScalK, ClusterReduce, true> m0(ptr, scal, red, c0);
        hoist_to_shared<PG, U>(m0, reinterpret_cast<float *>(stage_mem));
    }
    uint32_t s = 0;
    auto iterate = [&](auto guard_tag) {
        constexpr bool GUARD = decltype(guard_tag)::value;
        using MG = Machine<PG, U, PtrK, ScalK, ClusterReduce, GUARD, HOIST>;
        for (uint32_t row = first; row < P.rows; row += step) {
            Coords<U> ck;
            coords_of(row, ck);
            MG m(ptr, scal, red, ck);
            m.hoisted = hv;
            m.hoisted_shared = reinterpret_cast<const float *>(stage_mem);
            if (depth) {
                cp_async_wait(depth - 1);
                m.template stage_fetch<C_ROW_THREADS>(ring + s * STAGE);
                const uint32_t rn = row + depth * step;  // the stage just read is refilled with the row `depth` iterations ahead
                if (rn < P.rows) {
                    Coords<U> nx;
                    coords_of(rn, nx);
                    MG::template stage_issue<C_ROW_THREADS>(ptr, nx.flat0, nx.ok, stage0 + s * STAGE);
                }
                cp_async_commit();
                s = s + 1 == depth ? 0 : s + 1;
            } else {
                m.issue_loads();
            }
            m.run();
        }
    };
    if (full) iterate(FalseTag{});
    else iterate(TrueTag{});
    if (depth) cp_async_wait(0);
    // the next kernel of the stream may start only now: released at the top, its clusters took the places of this
    // kernel's retiring ones early and waited there, which measured 10-20 % slower back to back
    pdl_release();
    cluster_sync();
}

// A kernel that waits, bounded, for an mbarrier phase nothing completes: exercises the give-up path of
// mbar_wait_bounded and the status word without any copy in flight.
__global__ void lt_wait_probe(uint64_t limit_ns) {
    __shared__ __align__(8) uint64_t bar;
    const uint32_t b = (uint32_t)__cvta_generic_to_shared(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (!mbar_wait_bounded(b, 0, limit_ns) && threadIdx.x == 0) atomicOr(&lt_device_status, 1u);
}

}  // namespace
