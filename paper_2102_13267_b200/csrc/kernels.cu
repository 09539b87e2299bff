// Fused-group kernels for sm_100a: every thread interprets the group's register program
// (vm.h) on chunks of LT_VM_V consecutive elements.  Three shells share one interpreter:
//   lt_ew_kernel     elementwise / broadcast groups, grid-stride over chunks
//   lt_row_kernel    groups with row reductions: a power-of-two thread group owns a row,
//                    reduces with warp shuffles and, across warps, through shared memory
//   lt_multi_kernel  one program over many independent tensors (horizontal fusion)
// The program, pointer table and immediates arrive as a __grid_constant__ parameter and
// are read from the constant bank.  No tensor cores: nothing here is a contraction.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <cstddef>

#include "launch.h"
#include "pdl.cuh"
#include "vm.h"
#include "vm_core.inc"
#include "vm_ops.cuh"

namespace {

constexpr int V = LT_VM_V;
constexpr int NT = LT_VM_NT;  // R[0..NT-1] are the temporaries, R[NT] is ACC
static_assert(LT_VM_NT == 3 && LT_VM_ND == LT_VM_NT + 1, "the asm operand list below names three temporaries");

#ifndef LT_EW_MIN_BLOCKS
#define LT_EW_MIN_BLOCKS 3
#endif

struct Chunk {
    uint64_t flat0;  // flat index of lane 0
    uint32_t row;
    uint32_t col0;   // column of lane 0
    int nvalid;      // lanes 0..nvalid-1 exist
    bool row_ok;
};

struct RowCtx {
    float *smem;       // 2 x 32 floats
    uint32_t phase;
    uint32_t group;    // threads per row
    uint32_t warp, lane;
};

// ---------------------------------------------------------------- environments
struct EnvK {
    const LtKParams &P;
    __device__ __forceinline__ uint32_t scal(uint32_t i) const { return P.scal[i]; }
    __device__ __forceinline__ uint64_t ptr(uint32_t s) const { return P.ptr[s]; }
    __device__ __forceinline__ uint32_t dtype(uint32_t s) const { return P.io_dtype[s]; }
    __device__ __forceinline__ uint32_t cls(uint32_t s) const { return P.io_class[s]; }
    __device__ __forceinline__ uint32_t pitch(uint32_t s) const { return P.pitch[s]; }
};

struct EnvM {
    const LtMultiParams &P;
    uint32_t base;  // instance * n_slots
    __device__ __forceinline__ uint32_t scal(uint32_t i) const { return P.scal[i]; }
    __device__ __forceinline__ uint64_t ptr(uint32_t s) const { return P.ptr[base + s]; }
    __device__ __forceinline__ uint32_t dtype(uint32_t s) const { return P.io_dtype[s]; }
    __device__ __forceinline__ uint32_t cls(uint32_t) const { return LT_CLS_FULL; }
    __device__ __forceinline__ uint32_t pitch(uint32_t) const { return 0; }
};

// Random bits of the V lanes whose flat indices start at flat0 (element i uses word i mod 4 of
// block i / 4).  Kept out of line: its ten rounds would otherwise inflate the register budget of
// the whole interpreter.
__device__ __noinline__ void philox_chunk(uint32_t *out, uint64_t flat0, uint32_t k0, uint32_t k1, uint32_t o0,
                                          uint32_t o1) {
    const uint64_t q = flat0 >> 2;
    const uint32_t sh = (uint32_t)flat0 & 3u;
    uint32_t a[4], b[4];
    philox4x32_10((uint32_t)q, (uint32_t)(q >> 32), o0, o1, k0, k1, a);
    philox4x32_10((uint32_t)(q + 1), (uint32_t)((q + 1) >> 32), o0, o1, k0, k1, b);
    if (sh == 0) {
        out[0] = a[0]; out[1] = a[1]; out[2] = a[2]; out[3] = a[3];
        out[4] = b[0]; out[5] = b[1]; out[6] = b[2]; out[7] = b[3];
        return;
    }
    // chunk does not start on a block boundary (ragged rows): a third block covers the tail
    uint32_t c[4];
    philox4x32_10((uint32_t)(q + 2), (uint32_t)((q + 2) >> 32), o0, o1, k0, k1, c);
    const uint32_t w[12] = {a[0], a[1], a[2], a[3], b[0], b[1], b[2], b[3], c[0], c[1], c[2], c[3]};
    for (int i = 0; i < V; ++i) out[i] = w[i + sh];
}

// ------------------------------------------------------------------- memory
__device__ __forceinline__ uint32_t esz_log2(uint32_t dt) { return dt == LT_ST_BF16 ? 1u : (dt == LT_ST_U8 ? 0u : 2u); }

// ragged tail or unaligned pointer: element by element, packed into the same storage format
__device__ __noinline__ void load_raw_slow(float *d, const char *p, uint32_t dt, int nvalid) {
    if (dt == LT_ST_BF16) {
        const unsigned short *q = reinterpret_cast<const unsigned short *>(p);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t lo = 2 * j < nvalid ? q[2 * j] : 0u;
            uint32_t hi = 2 * j + 1 < nvalid ? q[2 * j + 1] : 0u;
            d[j] = u2f(lo | (hi << 16));
        }
    } else if (dt == LT_ST_U8) {
        const unsigned char *q = reinterpret_cast<const unsigned char *>(p);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            uint32_t w = 0;
#pragma unroll
            for (int b = 0; b < 4; ++b)
                if (4 * j + b < nvalid) w |= (uint32_t)q[4 * j + b] << (8 * b);
            d[j] = u2f(w);
        }
    } else {
        const float *q = reinterpret_cast<const float *>(p);
#pragma unroll
        for (int i = 0; i < V; ++i) d[i] = i < nvalid ? q[i] : 0.0f;
    }
}

// Raw chunk load: lanes keep the storage format (bf16: 4 packed words, u8: 2 packed words,
// 32-bit types: 8 words); CVT widens later so the load itself stays asynchronous.
template <class Env>
__device__ __forceinline__ void load_raw(float (&d)[V], const Env &E, uint32_t slot, const Chunk &ck) {
    const uint32_t dt = E.dtype(slot), cls = E.cls(slot);
    const char *base = reinterpret_cast<const char *>(E.ptr(slot));
    if (cls == LT_CLS_ROWVEC || cls == LT_CLS_SCALAR) {  // one element, replicated in storage format
        const uint64_t idx = cls == LT_CLS_ROWVEC ? (ck.row_ok ? ck.row : 0) : 0;
        if (dt == LT_ST_BF16) {
            uint32_t h = __ldg(reinterpret_cast<const unsigned short *>(base) + idx);
            h |= h << 16;
#pragma unroll
            for (int i = 0; i < 4; ++i) d[i] = u2f(h);
        } else if (dt == LT_ST_U8) {
            uint32_t b = __ldg(reinterpret_cast<const unsigned char *>(base) + idx) * 0x01010101u;
            d[0] = u2f(b);
            d[1] = u2f(b);
        } else {
            float x = __ldg(reinterpret_cast<const float *>(base) + idx);
#pragma unroll
            for (int i = 0; i < V; ++i) d[i] = x;
        }
        return;
    }
    const bool colvec = cls == LT_CLS_COLVEC;
    // (pitched: a slice of wider rows read in place -- row * pitch + column)
    const uint64_t idx = colvec ? (uint64_t)ck.col0 : cls == LT_CLS_PITCHED ? (uint64_t)(ck.row_ok ? ck.row : 0) * E.pitch(slot) + ck.col0 : ck.flat0;
    const char *p = base + (idx << esz_log2(dt));
    const uintptr_t need = dt == LT_ST_U8 ? 7u : 15u;
    if (ck.nvalid == V && (reinterpret_cast<uintptr_t>(p) & need) == 0) {
        if (dt == LT_ST_BF16) {
            uint4 a = colvec ? __ldg(reinterpret_cast<const uint4 *>(p)) : __ldcs(reinterpret_cast<const uint4 *>(p));
            d[0] = u2f(a.x); d[1] = u2f(a.y); d[2] = u2f(a.z); d[3] = u2f(a.w);
        } else if (dt == LT_ST_U8) {
            uint2 a = colvec ? __ldg(reinterpret_cast<const uint2 *>(p)) : __ldcs(reinterpret_cast<const uint2 *>(p));
            d[0] = u2f(a.x); d[1] = u2f(a.y);
        } else {
            const uint4 *q = reinterpret_cast<const uint4 *>(p);
            uint4 a = colvec ? __ldg(q) : __ldcs(q);
            uint4 b = colvec ? __ldg(q + 1) : __ldcs(q + 1);
            d[0] = u2f(a.x); d[1] = u2f(a.y); d[2] = u2f(a.z); d[3] = u2f(a.w);
            d[4] = u2f(b.x); d[5] = u2f(b.y); d[6] = u2f(b.z); d[7] = u2f(b.w);
        }
        return;
    }
    {
        // staged through a scratch array so the register-resident lanes never have their address taken
        float tmp[V];
        load_raw_slow(tmp, p, dt, ck.nvalid);
#pragma unroll
        for (int i = 0; i < V; ++i) d[i] = tmp[i];
    }
}

// raw chunk (storage format) -> 32-bit lanes
__device__ __forceinline__ void widen(float (&d)[V], uint32_t dt) {
    if (dt == LT_ST_BF16) {
        uint32_t w0 = f2u(d[0]), w1 = f2u(d[1]), w2 = f2u(d[2]), w3 = f2u(d[3]);
        d[0] = u2f(w0 << 16); d[1] = u2f(w0 & 0xffff0000u);
        d[2] = u2f(w1 << 16); d[3] = u2f(w1 & 0xffff0000u);
        d[4] = u2f(w2 << 16); d[5] = u2f(w2 & 0xffff0000u);
        d[6] = u2f(w3 << 16); d[7] = u2f(w3 & 0xffff0000u);
    } else if (dt == LT_ST_U8) {
        uint32_t w0 = f2u(d[0]), w1 = f2u(d[1]);
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            d[b] = u2f((w0 >> (8 * b)) & 0xffu);
            d[4 + b] = u2f((w1 >> (8 * b)) & 0xffu);
        }
    }
}

__device__ __noinline__ void store_chunk_slow(const float *a, char *p, uint32_t dt, int nvalid) {
    for (int i = 0; i < V; ++i) {
        if (i < nvalid) {
            if (dt == LT_ST_BF16) reinterpret_cast<__nv_bfloat16 *>(p)[i] = __float2bfloat16_rn(a[i]);
            else if (dt == LT_ST_U8) reinterpret_cast<unsigned char *>(p)[i] = (unsigned char)f2u(a[i]);
            else reinterpret_cast<float *>(p)[i] = a[i];
        }
    }
}

template <class Env>
__device__ __forceinline__ void store_chunk(const float (&a)[V], const Env &E, uint32_t slot, const Chunk &ck) {
    const uint32_t dt = E.dtype(slot), cls = E.cls(slot);
    char *base = reinterpret_cast<char *>(E.ptr(slot));
    if (cls == LT_CLS_ROWVEC) {  // one value per row, written by the thread that owns column 0
        if (ck.col0 == 0 && ck.row_ok) {
            if (dt == LT_ST_BF16) reinterpret_cast<__nv_bfloat16 *>(base)[ck.row] = __float2bfloat16_rn(a[0]);
            else if (dt == LT_ST_U8) reinterpret_cast<unsigned char *>(base)[ck.row] = (unsigned char)f2u(a[0]);
            else reinterpret_cast<float *>(base)[ck.row] = a[0];
        }
        return;
    }
    char *p = base + (ck.flat0 << esz_log2(dt));
    const uintptr_t need = dt == LT_ST_U8 ? 7u : 15u;
    if (ck.nvalid == V && (reinterpret_cast<uintptr_t>(p) & need) == 0) {
        if (dt == LT_ST_BF16) {
            uint4 w;
            __nv_bfloat162 h;
            h = __floats2bfloat162_rn(a[0], a[1]); w.x = *reinterpret_cast<uint32_t *>(&h);
            h = __floats2bfloat162_rn(a[2], a[3]); w.y = *reinterpret_cast<uint32_t *>(&h);
            h = __floats2bfloat162_rn(a[4], a[5]); w.z = *reinterpret_cast<uint32_t *>(&h);
            h = __floats2bfloat162_rn(a[6], a[7]); w.w = *reinterpret_cast<uint32_t *>(&h);
            __stcs(reinterpret_cast<uint4 *>(p), w);
        } else if (dt == LT_ST_U8) {
            uint2 w;
            w.x = (f2u(a[0]) & 0xffu) | ((f2u(a[1]) & 0xffu) << 8) | ((f2u(a[2]) & 0xffu) << 16) | (f2u(a[3]) << 24);
            w.y = (f2u(a[4]) & 0xffu) | ((f2u(a[5]) & 0xffu) << 8) | ((f2u(a[6]) & 0xffu) << 16) | (f2u(a[7]) << 24);
            __stcs(reinterpret_cast<uint2 *>(p), w);
        } else {
            uint4 w0 = make_uint4(f2u(a[0]), f2u(a[1]), f2u(a[2]), f2u(a[3]));
            uint4 w1 = make_uint4(f2u(a[4]), f2u(a[5]), f2u(a[6]), f2u(a[7]));
            __stcs(reinterpret_cast<uint4 *>(p), w0);
            __stcs(reinterpret_cast<uint4 *>(p) + 1, w1);
        }
        return;
    }
    {
        float tmp[V];
#pragma unroll
        for (int i = 0; i < V; ++i) tmp[i] = a[i];
        store_chunk_slow(tmp, p, dt, ck.nvalid);
    }
}

// ------------------------------------------------------------ row reductions
template <int KIND>
__device__ __forceinline__ float red_comb(float a, float b) {
    if constexpr (KIND == 0) return __fadd_rn(a, b);
    else if constexpr (KIND == 1) return max_nan(a, b);
    else return min_nan(a, b);
}

template <int KIND>
__device__ __forceinline__ void row_reduce(float (&acc)[V], const Chunk &ck, RowCtx *rc) {
    const float ident = KIND == 0 ? 0.0f : (KIND == 1 ? -INFINITY : INFINITY);
    float part = ident;
#pragma unroll
    for (int i = 0; i < V; ++i) part = red_comb<KIND>(part, i < ck.nvalid ? acc[i] : ident);
    const uint32_t width = rc->group < 32u ? rc->group : 32u;
    for (uint32_t off = width >> 1; off > 0; off >>= 1)
        part = red_comb<KIND>(part, __shfl_xor_sync(0xffffffffu, part, off));
    if (rc->group > 32u) {
        float *buf = rc->smem + (rc->phase & 1u) * 32u;
        rc->phase++;
        if (rc->lane == 0) buf[rc->warp] = part;
        __syncthreads();
        const uint32_t wpr = rc->group >> 5;
        const uint32_t first = (rc->warp / wpr) * wpr;
        part = buf[first];
        for (uint32_t w = 1; w < wpr; ++w) part = red_comb<KIND>(part, buf[first + w]);
    }
#pragma unroll
    for (int i = 0; i < V; ++i) acc[i] = part;
}

// -------------------------------------------------------------- interpreter
// Program, immediates and pointer table staged in shared memory, where the PTX core reads them
// with uniform (broadcast) loads.
struct Staged {
    LtIns ins[LT_VM_MAX_INS + 2];
    uint32_t scal[LT_VM_MAX_SCAL];
    uint64_t ptr[LT_VM_MAX_PTR];
    uint32_t soff[LT_VM_MAX_PTR];  // byte offset of the slot inside a staging buffer, 0xFFFFFFFF = not staged
    LtLoop loop;
    float red[64];
};
static_assert(offsetof(Staged, scal) == LT_VM_SM_SCAL && offsetof(Staged, ptr) == LT_VM_SM_PTR &&
                  offsetof(Staged, soff) == LT_VM_SM_SOFF && offsetof(Staged, loop) == LT_VM_SM_LOOP &&
                  offsetof(Staged, loop.stg) == LT_VM_SM_STG &&
                  offsetof(Staged, loop.pf_lo) == LT_VM_SM_STG + 16 * LT_VM_MAX_PTR &&
                  offsetof(Staged, red) == LT_VM_SM_RED,
              "the PTX core addresses these fields by constant offset");

// Pointer-table entry for the PTX core: bit 63 marks a slot whose chunks cannot use 128-bit accesses.
__device__ __forceinline__ uint64_t flag_pointer(uint64_t p, uint32_t dt, bool rows_aligned) {
    const uint64_t need = dt == LT_ST_U8 ? 7u : 15u;
    return ((p & need) == 0 && rows_aligned) ? p : (p | (1ull << 63));
}

__device__ __forceinline__ void lanes_of(const uint64_t (&p)[4], float (&f)[V]) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        f[2 * j] = u2f((uint32_t)p[j]);
        f[2 * j + 1] = u2f((uint32_t)(p[j] >> 32));
    }
}

__device__ __forceinline__ void pairs_of(const float (&f)[V], uint64_t (&p)[4]) {
#pragma unroll
    for (int j = 0; j < 4; ++j) p[j] = (uint64_t)f2u(f[2 * j]) | ((uint64_t)f2u(f[2 * j + 1]) << 32);
}

#define LT_VM_OPERANDS                                                                                              \
    : "+l"(R[NT][0]), "+l"(R[NT][1]), "+l"(R[NT][2]), "+l"(R[NT][3]), "+l"(R[0][0]), "+l"(R[0][1]), "+l"(R[0][2]),  \
      "+l"(R[0][3]), "+l"(R[1][0]), "+l"(R[1][1]), "+l"(R[1][2]), "+l"(R[1][3]), "+l"(R[2][0]), "+l"(R[2][1]),      \
      "+l"(R[2][2]), "+l"(R[2][3]), "+r"(pc), "=r"(eop), "=r"(eimm)                                                 \
      , "+r"(c), "+l"(off4), "+r"(coff4), "+r"(tail), "+r"(stg)                                                     \
    : "r"(smem_s)                                                                                                   \
    : "memory"

// Runs the group's program.  R[0..3] are T0..T3, R[4] is ACC.  The PTX core runs until an opcode it does
// not implement (see gen_vm_core.py); that opcode is executed here and the core re-entered.  With
// LtLoop::inloop set the core also walks the thread's chunks by itself and `chunk_of(c)` rebuilds the
// coordinates of chunk c for the code here; otherwise the call covers the one chunk given.
// Pointer slot an escaped load/store refers to: the immediate is the slot, except for staged forms,
// whose immediate is the slot's offset inside the staging buffer.
__device__ __forceinline__ uint32_t slot_of(const Staged &S, bool staged, uint32_t imm) {
    if (!staged) return imm;
    uint32_t s = 0;
    while (s + 1 < LT_VM_MAX_PTR && S.soff[s] != imm) ++s;
    return s;
}

// Executes one opcode the PTX core left to C++ (see gen_vm_core.py).  Out of line, with the machine state
// handed over in memory: these paths are cold (ragged or unaligned chunks, irregular rows, math-library
// transcendentals), and inlined they would raise the register count of the whole kernel by a third.
// r[4 * k .. 4 * k + 3] is T[k] for k < NT and ACC for k = NT.
template <bool ROW, class Env>
__device__ __noinline__ void handle_escape(uint64_t *r, uint32_t eop, uint32_t eimm, const Env &E, const Chunk &ck, RowCtx *rc,
                                           const Staged &S) {
    float f[V];
    uint64_t(&acc)[4] = *reinterpret_cast<uint64_t(*)[4]>(r + 4 * NT);
    const bool is_ld = eop >= OP_LD && eop < OP_STG;
    const bool is_f2m = eop >= OP_F2M && eop < OP_F2;
    if (is_ld || is_f2m) {
        // a load that was not linked to a vector path (unaligned pointer, broadcast class), or one
        // that met a ragged chunk: element-wise load, then widen
        const bool staged = (eop >= OP_LDS && eop < OP_STG) || eop >= OP_F2MS;
        const uint32_t slot = slot_of(S, staged, eimm);
        load_raw(f, E, slot, ck);
        widen(f, E.dtype(slot));
        if (is_ld) {
            const uint32_t d = eop < OP_LDG ? eop - OP_LD : eop < OP_LDS ? (eop - OP_LDG) % LT_VM_ND : (eop - OP_LDS) % LT_VM_ND;
            pairs_of(f, *reinterpret_cast<uint64_t(*)[4]>(r + 4 * d));
        } else {
            const uint32_t k = eop < OP_F2MG ? eop - OP_F2M : eop < OP_F2MS ? (eop - OP_F2MG) / 6u : (eop - OP_F2MS) / 3u;
            float a[V];
            lanes_of(acc, a);
#pragma unroll
            for (int i = 0; i < V; ++i)
                a[i] = k == F2M_ADD ? __fadd_rn(a[i], f[i]) : k == F2M_SUB ? __fsub_rn(a[i], f[i])
                     : k == F2M_RSUB ? __fsub_rn(f[i], a[i]) : __fmul_rn(a[i], f[i]);
            pairs_of(a, acc);
        }
        return;
    }
    lanes_of(acc, f);
    if (eop == OP_ST || (eop >= OP_STG && eop < OP_STG + 3)) {
        store_chunk(f, E, eimm, ck);
        return;
    }
    if (eop == OP_IOTA_ROW) {
        const uint32_t row = (ck.row / E.scal(eimm)) % E.scal(eimm + 1);
#pragma unroll
        for (int i = 0; i < V; ++i) f[i] = u2f(row);
    } else if (eop == OP_PHILOX) {
        uint32_t w[V];
        philox_chunk(w, ck.flat0, E.scal(eimm), E.scal(eimm + 1), E.scal(eimm + 2), E.scal(eimm + 3));
#pragma unroll
        for (int i = 0; i < V; ++i) f[i] = u2f(w[i]);
    } else if (eop >= OP_RED_SUM && eop <= OP_RED_MIN) {
        if constexpr (ROW) {
            if (eop == OP_RED_SUM) row_reduce<0>(f, ck, rc);
            else if (eop == OP_RED_MAX) row_reduce<1>(f, ck, rc);
            else row_reduce<2>(f, ck, rc);
        }
    } else {  // correctly rounded transcendentals of the precise flavour
#pragma unroll
        for (int i = 0; i < V; ++i) {
            if (eop == OP_U_EXP) f[i] = un<OP_U_EXP, false>(f[i]);
            else if (eop == OP_U_LOG) f[i] = un<OP_U_LOG, false>(f[i]);
            else if (eop == OP_U_TANH) f[i] = un<OP_U_TANH, false>(f[i]);
            else if (eop == OP_U_SIGMOID) f[i] = un<OP_U_SIGMOID, false>(f[i]);
            else if (eop == OP_U_GELU) f[i] = un<OP_U_GELU, false>(f[i]);
        }
    }
    pairs_of(f, acc);
}

// Runs the group's program.  R[0..NT-1] are the temporaries, R[NT] is ACC.  The PTX core runs until an opcode
// it does not implement; that opcode is executed by handle_escape and the core re-entered.  With
// LtLoop::inloop set the core also walks the thread's chunks by itself and `chunk_of(c)` rebuilds the
// coordinates of chunk c for the escape code; otherwise the call covers the one chunk given.
template <int FLAV, bool ROW, class Env, class ChunkOf>
__device__ __forceinline__ void run_program(const Env &E, ChunkOf chunk_of, uint32_t c, const Chunk &first, RowCtx *rc,
                                            const Staged &S, uint32_t stg, uint32_t flags = 0) {
    const uint32_t smem_s = (uint32_t)__cvta_generic_to_shared(&S);
    uint64_t R[NT + 1][4];  // not initialised: a program writes every register before it reads it
    uint32_t pc = smem_s;
    uint64_t off4 = first.flat0 << 2;
    uint32_t coff4 = first.col0 << 2;
    uint32_t tail = (first.nvalid != V ? 1u : 0u) | flags;  // see entry_code() in gen_vm_core.py for the bits
#pragma unroll 1
    for (;;) {
        uint32_t eop, eimm;
        if constexpr (FLAV == 0) asm volatile(LT_VM_CORE_FAST LT_VM_OPERANDS);
        else if constexpr (FLAV == 1) asm volatile(LT_VM_CORE_PRECISE LT_VM_OPERANDS);
        else asm volatile(LT_VM_CORE_IEEE LT_VM_OPERANDS);
        if (eop == OP_END) break;
        uint64_t spill[4 * (NT + 1)];  // the state travels through memory so that it never has its address taken
#pragma unroll
        for (int k = 0; k <= NT; ++k)
#pragma unroll
            for (int j = 0; j < 4; ++j) spill[4 * k + j] = R[k][j];
        const Chunk ck = chunk_of(c);
        handle_escape<ROW>(spill, eop, eimm, E, ck, rc, S);
#pragma unroll
        for (int k = 0; k <= NT; ++k)
#pragma unroll
            for (int j = 0; j < 4; ++j) R[k][j] = spill[4 * k + j];
    }
}

template <class P>
__device__ __forceinline__ void stage_program(Staged &S, const P &prm) {
    for (uint32_t i = threadIdx.x; i < prm.n_ins + 2; i += blockDim.x) {
        LtIns in;
        in.op = OP_END;
        in.imm = 0;
        if (i < prm.n_ins) in = prm.ins[i];
        S.ins[i] = in;
    }
    for (uint32_t i = threadIdx.x; i < LT_VM_MAX_SCAL; i += blockDim.x) S.scal[i] = prm.scal[i];
    if (threadIdx.x < LT_VM_MAX_PTR) S.soff[threadIdx.x] = 0xffffffffu;
    if (threadIdx.x < sizeof(LtLoop) / 4) reinterpret_cast<uint32_t *>(&S.loop)[threadIdx.x] = 0;
}

// Link step: rewrites the generic load / store / memory-operand opcodes of the staged program into the
// vector-path forms this launch's pointers allow (see vm.h).  S.ptr (bit 63 = no vector path) and S.soff
// must be final.  `all_slots_ok` false keeps everything generic.
__device__ __forceinline__ void link_program(Staged &S, uint32_t n_ins, const uint8_t *io_dtype, const uint8_t *io_class,
                                             bool multi) {
    for (uint32_t i = threadIdx.x; i < n_ins; i += blockDim.x) {
        LtIns in = S.ins[i];
        const uint32_t op = in.op, slot = in.imm;
        const bool ld = op >= OP_LD && op < OP_LD + LT_VM_ND, st = op == OP_ST, f2m = op >= OP_F2M && op < OP_F2M + F2M_COUNT;
        if (!(ld || st || f2m)) continue;
        const uint32_t dt = io_dtype[slot], cls = multi ? (uint32_t)LT_CLS_FULL : (uint32_t)io_class[slot];
        if ((S.ptr[slot] >> 63) || cls > LT_CLS_COLVEC) continue;
        const uint32_t sz = dt == LT_ST_BF16 ? 1u : dt == LT_ST_U8 ? 2u : 0u;
        const bool staged = S.soff[slot] != 0xffffffffu;
        if (ld) {
            const uint32_t d = op - OP_LD;
            if (staged) { in.op = OP_LDS + sz * LT_VM_ND + d; in.imm = S.soff[slot]; }
            else in.op = OP_LDG + (sz * 2 + cls) * LT_VM_ND + d;
        } else if (f2m) {
            const uint32_t k = op - OP_F2M;
            if (staged) { in.op = OP_F2MS + k * 3 + sz; in.imm = S.soff[slot]; }
            else in.op = OP_F2MG + (k * 3 + sz) * 2 + cls;
        } else if (cls == LT_CLS_FULL) {
            in.op = OP_STG + sz;
        }
        S.ins[i] = in;
    }
}

// Asynchronous 16-byte (or 8-byte) copy global -> shared; completion is tracked per thread in groups.
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

// Starts the copies of one future chunk (first element e0) of every staged input into staging buffer `buf`.
__device__ __forceinline__ void stage_chunk(const LtLoop &lp, uint64_t e0, uint32_t buf) {
    const uint32_t total = (lp.stg_n & 0xffu) + ((lp.stg_n >> 8) & 0xffu) + ((lp.stg_n >> 16) & 0xffu);  // counts per element size
#pragma unroll 1
    for (uint32_t k = 0; k < total && k < LT_VM_MAX_PTR; ++k) {
        const uint32_t sh = lp.stg[k].shift;
        const char *src = reinterpret_cast<const char *>(((uint64_t)lp.stg[k].ptr_hi << 32) | lp.stg[k].ptr_lo) + (e0 << sh);
        const uint32_t dst = buf + lp.stg[k].dst;
        if (sh == 0) cp_async8(dst, src);
        else {
            cp_async16(dst, src);
            if (sh == 2) cp_async16(dst + LT_VM_STAGE_PIECE, src + 16);
        }
    }
}

// Builds LtLoop::stg: the staged inputs sorted by element size (4-, 2-, 1-byte), counts packed in stg_n.
template <class PtrOf>
__device__ __forceinline__ void fill_stage_list(LtLoop &lp, const uint8_t *io_stage, const uint8_t *io_dtype, uint32_t n_slots,
                                                PtrOf ptr_of) {
    uint32_t k = 0, counts = 0;
    for (uint32_t pass = 0; pass < 3; ++pass) {  // pass 0: 4-byte elements, 1: 2-byte, 2: 1-byte
        uint32_t n = 0;
        for (uint32_t s = 0; s < n_slots; ++s) {
            if (io_stage[s] == 0xffu) continue;
            const uint32_t sz = io_dtype[s] == LT_ST_BF16 ? 1u : io_dtype[s] == LT_ST_U8 ? 2u : 0u;
            if (sz != pass) continue;
            const uint64_t p = ptr_of(s);
            lp.stg[k].ptr_lo = (uint32_t)p;
            lp.stg[k].ptr_hi = (uint32_t)(p >> 32);
            lp.stg[k].dst = io_stage[s] * LT_VM_STAGE_PIECE;
            lp.stg[k].shift = 2u - sz;
            ++k;
            ++n;
        }
        counts |= n << (8 * pass);
    }
    lp.stg_n = counts;
}

// Fills the loop constants shared by the elementwise and row kernels (thread 0, before the link step).
__device__ __forceinline__ void fill_loop(LtLoop &lp, const LtKParams &P, uint32_t mode, uint32_t stride, uint32_t n_iter,
                                          uint64_t step4, uint32_t stage_base, bool prefetch) {
    const uint32_t depth = P.stage_depth;
    lp.stride = stride;
    lp.n_chunks = n_iter;
    lp.body_off = P.n_pro * (uint32_t)sizeof(LtIns);
    lp.depth = depth;
    lp.buf_bytes = P.stage_pieces * LT_VM_STAGE_PIECE;
    lp.buf_total = depth * lp.buf_bytes;
    lp.stage_base = stage_base;
    // bit 8: L2 prefetch by the loads (no staging); bit 9: L2 prefetch behind a short staging ring
    lp.inloop = mode | ((prefetch && !depth) ? 256u : 0u) | ((depth && depth < 3) ? 512u : 0u);
    lp.rowcol = P.rowcol;
    lp.cpr = P.cpr;
    lp.div_mul = P.div_mul;
    lp.div_sh1 = P.div_sh1;
    lp.div_sh2 = P.div_sh2;
    lp.cols = P.cols;
    lp.prefetch = (prefetch && !depth) ? 1u : 0u;  // without staging, pull the next chunk into L2 instead
    lp.pf_lo = (uint32_t)step4;
    lp.pf_hi = (uint32_t)(step4 >> 32);
    lp.n4_lo = (uint32_t)(P.n * 4);
    lp.n4_hi = (uint32_t)((P.n * 4) >> 32);
    lp.group = P.group;
    // row-wise opcodes run inside the core when every thread of a row group owns a complete chunk
    const bool regular = (P.cols % V) == 0 && (mode != 2 || P.group * V == P.cols);
    lp.inline_rows = (regular && P.n < (1ull << 32)) ? 1u : 0u;
    const uint64_t dpf = (uint64_t)depth * step4;
    lp.dpf_lo = (uint32_t)dpf;
    lp.dpf_hi = (uint32_t)(dpf >> 32);
    lp.stg_n = 0;
    if (depth) fill_stage_list(lp, P.io_stage, P.io_dtype, LT_VM_MAX_PTR, [&P](uint32_t s) { return P.ptr[s]; });
}

__device__ __forceinline__ Chunk ew_chunk(const LtKParams &P, uint32_t c) {
    Chunk ck;
    ck.row_ok = true;
    if (!P.rowcol) {
        ck.flat0 = (uint64_t)c * V;
        ck.row = 0;
        ck.col0 = c * V;
        const uint64_t rem = P.n - ck.flat0;
        ck.nvalid = rem < (uint64_t)V ? (int)rem : V;
    } else {
        const uint32_t t = __umulhi(P.div_mul, c);
        const uint32_t row = (t + ((c - t) >> P.div_sh1)) >> P.div_sh2;
        const uint32_t cc = c - row * P.cpr;
        ck.row = row;
        ck.col0 = cc * V;
        ck.flat0 = (uint64_t)row * P.cols + ck.col0;
        const uint32_t rem = P.cols - ck.col0;
        ck.nvalid = rem < (uint32_t)V ? (int)rem : V;
    }
    return ck;
}

// ------------------------------------------------------------------ kernels
template <int FLAV>
__global__ void __launch_bounds__(LT_EW_THREADS, LT_EW_MIN_BLOCKS) lt_ew_kernel(const __grid_constant__ LtKParams P) {
    pdl_release();
    __shared__ __align__(16) Staged S;
    extern __shared__ __align__(16) unsigned char stage_mem[];
    const EnvK E{P};
    stage_program(S, P);
    __syncthreads();
    const bool linear = !P.rowcol || (P.cols % V) == 0;  // chunk c starts at element 8c
    const uint32_t stride = gridDim.x * blockDim.x;
    const uint32_t n_chunks = (uint32_t)P.n_chunks;      // the planner keeps chunk counts below 2^32 - stride
    const uint32_t depth = P.stage_depth;
    const uint32_t buf_bytes = P.stage_pieces * LT_VM_STAGE_PIECE;
    const uint32_t stage_base = (uint32_t)__cvta_generic_to_shared(stage_mem);
    if (threadIdx.x < LT_VM_MAX_PTR) {
        S.ptr[threadIdx.x] = flag_pointer(P.ptr[threadIdx.x], P.io_dtype[threadIdx.x], linear);
        if (depth && P.io_stage[threadIdx.x] != 0xffu) S.soff[threadIdx.x] = P.io_stage[threadIdx.x] * LT_VM_STAGE_PIECE;
    }
    // rows that are a multiple of the chunk and a chunk stride that is a multiple of the chunks per row: a
    // thread's next chunk is a fixed distance ahead in the same columns, no coordinates to recompute
    const bool fixed_cols = P.rowcol && linear && (stride % P.cpr) == 0;
    if (threadIdx.x == 0)
        fill_loop(S.loop, P, fixed_cols ? 2 : 1, stride, n_chunks, (uint64_t)stride * (V * 4), stage_base, linear);
    __syncthreads();
    link_program(S, P.n_ins, P.io_dtype, P.io_class, false);
    __syncthreads();
    pdl_wait();  // everything above read only the parameter block
    const uint32_t c0 = blockIdx.x * blockDim.x + threadIdx.x;
    if (c0 >= n_chunks) return;
    // Software pipeline: the full-class inputs of the thread's next `depth` chunks are in flight as
    // asynchronous copies into per-thread staging buffers while the current chunk is interpreted.
    const uint32_t buf0 = stage_base + threadIdx.x * 16u;
    if (depth) {
        uint64_t c = c0;
        for (uint32_t d = 0; d < depth; ++d) {
            if (c < P.n / V) stage_chunk(S.loop, c * V, buf0 + d * buf_bytes);
            cp_async_commit();
            c += stride;
        }
        cp_async_wait(depth - 1);
    }
    run_program<FLAV, false>(E, [&P](uint32_t c) { return ew_chunk(P, c); }, c0, ew_chunk(P, c0), nullptr, S, buf0);
    if (depth) cp_async_wait(0);
}

template <int FLAV, int MAXT>
__global__ void __launch_bounds__(MAXT, MAXT == 256 ? LT_EW_MIN_BLOCKS : 1) lt_row_kernel(const __grid_constant__ LtKParams P) {
    pdl_release();
    __shared__ __align__(16) Staged S;
    extern __shared__ __align__(16) unsigned char stage_mem[];
    const EnvK E{P};
    stage_program(S, P);
    __syncthreads();
    const uint32_t row_blocks = (P.rows + P.rows_per_cta - 1u) / P.rows_per_cta;
    const bool aligned_rows = (P.cols % V) == 0;
    const uint32_t depth = P.stage_depth;
    const uint32_t buf_bytes = P.stage_pieces * LT_VM_STAGE_PIECE;
    const uint32_t stage_base = (uint32_t)__cvta_generic_to_shared(stage_mem);
    const uint64_t step = (uint64_t)gridDim.x * P.rows_per_cta * P.cols;  // elements between a thread's iterations
    if (threadIdx.x < LT_VM_MAX_PTR) {
        S.ptr[threadIdx.x] = flag_pointer(P.ptr[threadIdx.x], P.io_dtype[threadIdx.x], aligned_rows);
        if (depth && P.io_stage[threadIdx.x] != 0xffu) S.soff[threadIdx.x] = P.io_stage[threadIdx.x] * LT_VM_STAGE_PIECE;
    }
    if (threadIdx.x == 0) fill_loop(S.loop, P, 2, gridDim.x, row_blocks, step * 4, stage_base, aligned_rows);
    __syncthreads();
    link_program(S, P.n_ins, P.io_dtype, P.io_class, false);
    __syncthreads();
    pdl_wait();  // everything above read only the parameter block
    RowCtx rc;
    rc.smem = S.red;
    rc.phase = 0;
    rc.group = P.group;
    rc.warp = threadIdx.x >> 5;
    rc.lane = threadIdx.x & 31u;
    const uint32_t sub = threadIdx.x >> P.group_log2;           // which row of this CTA's block of rows
    const uint32_t gl = threadIdx.x & (P.group - 1u);           // lane within the row's thread group
    // every thread of the CTA runs the same number of iterations (row reductions synchronise the CTA)
    auto chunk_of = [&P, sub, gl](uint32_t rb) {
        Chunk ck;
        ck.row = rb * P.rows_per_cta + sub;
        ck.row_ok = ck.row < P.rows;
        ck.col0 = gl * V;
        ck.flat0 = (uint64_t)ck.row * P.cols + ck.col0;
        int nv = 0;
        if (ck.row_ok && ck.col0 < P.cols) {
            const uint32_t rem = P.cols - ck.col0;
            nv = rem < (uint32_t)V ? (int)rem : V;
        }
        ck.nvalid = nv;
        return ck;
    };
    if (blockIdx.x >= row_blocks) return;
    const Chunk first = chunk_of(blockIdx.x);
    const bool col_full = gl * V + V <= P.cols;
    const uint32_t buf0 = stage_base + threadIdx.x * 16u;
    if (depth) {
        uint64_t e = first.flat0;
        for (uint32_t d = 0; d < depth; ++d) {
            if (col_full && e + V <= P.n) stage_chunk(S.loop, e, buf0 + d * buf_bytes);
            cp_async_commit();
            e += step;
        }
        cp_async_wait(depth - 1);
    }
    run_program<FLAV, true>(E, chunk_of, blockIdx.x, first, &rc, S, buf0, col_full ? 0u : 2u);
    if (depth) cp_async_wait(0);
}

template <int FLAV>
__global__ void __launch_bounds__(LT_EW_THREADS, LT_EW_MIN_BLOCKS) lt_multi_kernel(const __grid_constant__ LtMultiParams P) {
    pdl_release();
    __shared__ __align__(16) Staged S;
    extern __shared__ __align__(16) unsigned char stage_mem[];
    stage_program(S, P);
    if (threadIdx.x < LT_VM_MAX_PTR) {
        S.ptr[threadIdx.x] = 0;
        if (P.stage_depth && P.io_stage[threadIdx.x] != 0xffu) S.soff[threadIdx.x] = P.io_stage[threadIdx.x] * LT_VM_STAGE_PIECE;
    }
    __syncthreads();
    // linked once for all instances; an instance with an unaligned pointer has that slot flagged below and
    // its accesses leave the vector path at run time (staged slots are aligned in every instance)
    link_program(S, P.n_ins, P.io_dtype, nullptr, true);
    const uint32_t depth = P.stage_depth;
    const uint32_t buf_bytes = P.stage_pieces * LT_VM_STAGE_PIECE;
    const uint32_t stage_base = (uint32_t)__cvta_generic_to_shared(stage_mem);
    const uint32_t buf0 = stage_base + threadIdx.x * 16u;
    pdl_wait();  // everything above read only the parameter block
    for (uint32_t sc = blockIdx.x; sc < P.total_super; sc += gridDim.x) {
        // instance that owns super-chunk sc: last i with super_prefix[i] <= sc
        uint32_t lo = 0, hi = P.n_inst;
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (P.super_prefix[mid] <= sc) lo = mid; else hi = mid;
        }
        const EnvM E{P, lo * P.n_slots};
        const uint32_t numel = P.numel[lo];
        // within the instance the super-chunk is a flat range of chunks, walked by the core with stride 256
        const uint32_t chunk_first = (sc - P.super_prefix[lo]) * (LT_EW_THREADS * LT_MULTI_SUB);
        const uint32_t chunks_all = (numel + V - 1) / V;
        const uint32_t chunk_end = min(chunk_first + LT_EW_THREADS * LT_MULTI_SUB, chunks_all);
        __syncthreads();  // the previous super-chunk's tables are no longer in use
        if (threadIdx.x < P.n_slots) S.ptr[threadIdx.x] = flag_pointer(E.ptr(threadIdx.x), P.io_dtype[threadIdx.x], true);
        if (threadIdx.x == 32) {
            LtLoop &lp = S.loop;
            lp.stride = LT_EW_THREADS;
            lp.n_chunks = chunk_end;
            lp.depth = depth;
            lp.buf_bytes = buf_bytes;
            lp.buf_total = depth * buf_bytes;
            lp.stage_base = stage_base;
            lp.inloop = 1u | (depth ? 0u : 256u) | ((depth && depth < 3) ? 512u : 0u);
            lp.rowcol = 0;
            lp.prefetch = depth ? 0u : 1u;
            lp.pf_lo = LT_EW_THREADS * V * 4;
            lp.pf_hi = 0;
            lp.dpf_lo = depth * LT_EW_THREADS * V * 4;
            lp.dpf_hi = 0;
            lp.n4_lo = numel * 4u;
            lp.n4_hi = numel >> 30;
            lp.stg_n = 0;
            if (depth) fill_stage_list(lp, P.io_stage, P.io_dtype, P.n_slots, [&E](uint32_t s) { return E.ptr(s); });
        }
        __syncthreads();
        const uint32_t c0 = chunk_first + threadIdx.x;
        if (c0 < chunk_end) {
            if (depth) {
                uint32_t c = c0;
                for (uint32_t d = 0; d < depth; ++d) {
                    if ((uint64_t)c * V + V <= numel) stage_chunk(S.loop, (uint64_t)c * V, buf0 + d * buf_bytes);
                    cp_async_commit();
                    c += LT_EW_THREADS;
                }
                cp_async_wait(depth - 1);
            }
            auto chunk_of = [numel](uint32_t c) {
                Chunk ck;
                ck.flat0 = (uint64_t)c * V;
                ck.row = 0;
                ck.col0 = c * V;
                ck.row_ok = true;
                const uint32_t rem = numel - c * V;
                ck.nvalid = rem < (uint32_t)V ? (int)rem : V;
                return ck;
            };
            run_program<FLAV, false>(E, chunk_of, c0, chunk_of(c0), nullptr, S, buf0);
            if (depth) cp_async_wait(0);
        }
    }
}

}  // namespace

cudaError_t lt_launch_ew(const LtKParams &p, int flavour, unsigned grid, cudaStream_t stream) {
    const size_t dyn = (size_t)p.stage_depth * p.stage_pieces * LT_VM_STAGE_PIECE;
    if (flavour == 0) return launch_pdl(lt_ew_kernel<0>, grid, LT_EW_THREADS, dyn, stream, p);
    else if (flavour == 1) return launch_pdl(lt_ew_kernel<1>, grid, LT_EW_THREADS, dyn, stream, p);
    return launch_pdl(lt_ew_kernel<2>, grid, LT_EW_THREADS, dyn, stream, p);
}

cudaError_t lt_kernel_setup(size_t max_stage_bytes) {
    cudaError_t e = cudaFuncSetAttribute(lt_ew_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_stage_bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(lt_ew_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_stage_bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(lt_ew_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_stage_bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(lt_multi_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_stage_bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(lt_multi_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_stage_bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(lt_multi_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_stage_bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(lt_row_kernel<0, 256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_stage_bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(lt_row_kernel<1, 256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_stage_bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(lt_row_kernel<2, 256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_stage_bytes);
    return e;
}

cudaError_t lt_launch_row(const LtKParams &p, int flavour, unsigned grid, unsigned threads, cudaStream_t stream) {
    const size_t dyn = (size_t)p.stage_depth * p.stage_pieces * LT_VM_STAGE_PIECE;
    if (threads <= 256) {
        if (flavour == 0) return launch_pdl(lt_row_kernel<0, 256>, grid, threads, dyn, stream, p);
        else if (flavour == 1) return launch_pdl(lt_row_kernel<1, 256>, grid, threads, dyn, stream, p);
        return launch_pdl(lt_row_kernel<2, 256>, grid, threads, dyn, stream, p);
    }
    if (flavour == 0) return launch_pdl(lt_row_kernel<0, 1024>, grid, threads, (size_t)0, stream, p);
    else if (flavour == 1) return launch_pdl(lt_row_kernel<1, 1024>, grid, threads, (size_t)0, stream, p);
    return launch_pdl(lt_row_kernel<2, 1024>, grid, threads, (size_t)0, stream, p);
}

cudaError_t lt_launch_multi(const LtMultiParams &p, int flavour, unsigned grid, cudaStream_t stream) {
    const size_t dyn = (size_t)p.stage_depth * p.stage_pieces * LT_VM_STAGE_PIECE;
    if (flavour == 0) return launch_pdl(lt_multi_kernel<0>, grid, LT_EW_THREADS, dyn, stream, p);
    else if (flavour == 1) return launch_pdl(lt_multi_kernel<1>, grid, LT_EW_THREADS, dyn, stream, p);
    return launch_pdl(lt_multi_kernel<2>, grid, LT_EW_THREADS, dyn, stream, p);
}

cudaError_t lt_kernel_occupancy(int *ew_blocks_per_sm, int *row_blocks_per_sm_256, int *multi_blocks_per_sm) {
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(ew_blocks_per_sm, lt_ew_kernel<1>, LT_EW_THREADS, 0);
    if (e != cudaSuccess) return e;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(row_blocks_per_sm_256, lt_row_kernel<1, 256>, 256, 0);
    if (e != cudaSuccess) return e;
    return cudaOccupancyMaxActiveBlocksPerMultiprocessor(multi_blocks_per_sm, lt_multi_kernel<1>, LT_EW_THREADS, 0);
}
