// Reductions that run as kernels of their own instead of register programs: over the columns of a
// matrix (every dimension but the last), over a whole tensor, and over rows too long for a row's
// thread group to keep in registers when the surrounding program has no fused kernel for that length.
// All three read their input once with coalesced accesses, accumulate sums in binary64 (one rounding
// to the result's dtype at the end) and propagate NaN through max / min.  The column and whole-tensor
// forms run in two stages through a small array of binary64 partial results in scratch memory.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "launch.h"
#include "pdl.cuh"

namespace {

constexpr int RT = 256;  // threads per CTA

template <int KIND>
__device__ __forceinline__ double ident() {
    return KIND == 0 ? 0.0 : (KIND == 1 ? -INFINITY : INFINITY);
}

template <int KIND>
__device__ __forceinline__ double comb(double a, double b) {
    if constexpr (KIND == 0) return a + b;
    else if constexpr (KIND == 1) return (a != a || b != b) ? NAN : (a > b ? a : b);
    else return (a != a || b != b) ? NAN : (a < b ? a : b);
}

// element i of an array of storage dtype DT (0 f32, 1 bf16, 5 binary64 partials) as binary64
template <int DT>
__device__ __forceinline__ double load_as_double(const void *p, uint64_t i) {
    if constexpr (DT == 0) return (double)__ldg(reinterpret_cast<const float *>(p) + i);
    else if constexpr (DT == 1) return (double)__uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short *>(p) + i) << 16);
    else return reinterpret_cast<const double *>(p)[i];
}

template <int DT>
__device__ __forceinline__ void store_from_double(void *p, uint64_t i, double v) {
    if constexpr (DT == 0) reinterpret_cast<float *>(p)[i] = (float)v;
    else if constexpr (DT == 1) reinterpret_cast<__nv_bfloat16 *>(p)[i] = __float2bfloat16_rn((float)v);
    else reinterpret_cast<double *>(p)[i] = v;
}

template <int KIND>
__device__ __forceinline__ double cta_reduce(double v, double *smem) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v = comb<KIND>(v, __shfl_xor_sync(0xffffffffu, v, off));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();  // smem may still be read from a previous call
    if (lane == 0) smem[warp] = v;
    __syncthreads();
    double r = smem[0];
    for (int w = 1; w < RT / 32; ++w) r = comb<KIND>(r, smem[w]);
    return r;
}

// One CTA per row at a time; out[row] = reduce(in[row, :]).
template <int DT, int KIND>
__global__ void __launch_bounds__(RT) lt_reduce_rows(const void *in, void *out, uint32_t rows, uint64_t cols) {
    __shared__ double smem[RT / 32];
    pdl_release();
    pdl_wait();
    for (uint32_t r = blockIdx.x; r < rows; r += gridDim.x) {
        const uint64_t base = (uint64_t)r * cols;
        double a0 = ident<KIND>(), a1 = ident<KIND>();
        uint64_t c = threadIdx.x;
        for (; c + RT < cols; c += 2 * RT) {
            a0 = comb<KIND>(a0, load_as_double<DT>(in, base + c));
            a1 = comb<KIND>(a1, load_as_double<DT>(in, base + c + RT));
        }
        if (c < cols) a0 = comb<KIND>(a0, load_as_double<DT>(in, base + c));
        const double v = cta_reduce<KIND>(comb<KIND>(a0, a1), smem);
        if (threadIdx.x == 0) store_from_double<DT>(out, r, v);
    }
}

// W consecutive elements starting at element i (W = 4: i is a multiple of 4 and the array 16-byte aligned)
template <int DT, int W>
__device__ __forceinline__ void load_vec(const void *p, uint64_t i, double (&v)[W]) {
    if constexpr (W == 1) {
        v[0] = load_as_double<DT>(p, i);
    } else if constexpr (DT == 0) {
        const float4 f = __ldg(reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(p) + i));
        v[0] = f.x, v[1] = f.y, v[2] = f.z, v[3] = f.w;
    } else if constexpr (DT == 1) {
        const uint2 w = __ldg(reinterpret_cast<const uint2 *>(reinterpret_cast<const unsigned short *>(p) + i));
        v[0] = __uint_as_float(w.x << 16), v[1] = __uint_as_float(w.x & 0xffff0000u);
        v[2] = __uint_as_float(w.y << 16), v[3] = __uint_as_float(w.y & 0xffff0000u);
    } else {
        const double2 a = reinterpret_cast<const double2 *>(reinterpret_cast<const double *>(p) + i)[0];
        const double2 b = reinterpret_cast<const double2 *>(reinterpret_cast<const double *>(p) + i)[1];
        v[0] = a.x, v[1] = a.y, v[2] = b.x, v[3] = b.y;
    }
}

// Column reduction, one stage: CTA (bx, by) reduces rows [by * rows_per, ...) of the 32 * W columns bx * 32 * W ..;
// thread (x, y) of the 32 x 8 CTA owns W adjacent columns and walks rows y, y + 8, ...  The result goes to
// dst[by * cols + col].  W = 4 needs cols % 4 == 0 and a 16-byte aligned input.
template <int DT_IN, int DT_OUT, int KIND, int W>
__global__ void __launch_bounds__(RT) lt_reduce_cols(const void *in, void *dst, uint64_t rows, uint64_t cols, uint64_t rows_per) {
    __shared__ double smem[8][32 * W + 1];
    pdl_release();
    pdl_wait();
    const uint32_t x = threadIdx.x & 31u, y = threadIdx.x >> 5;
    const uint64_t col = ((uint64_t)blockIdx.x * 32u + x) * W;
    const uint64_t r0 = (uint64_t)blockIdx.y * rows_per;
    const uint64_t r1 = r0 + rows_per < rows ? r0 + rows_per : rows;
    double a0[W], a1[W];
#pragma unroll
    for (int w = 0; w < W; ++w) a0[w] = a1[w] = ident<KIND>();
    if (col < cols) {
        uint64_t r = r0 + y;
        for (; r + 8 < r1; r += 16) {
            double v0[W], v1[W];
            load_vec<DT_IN, W>(in, r * cols + col, v0);
            load_vec<DT_IN, W>(in, (r + 8) * cols + col, v1);
#pragma unroll
            for (int w = 0; w < W; ++w) a0[w] = comb<KIND>(a0[w], v0[w]), a1[w] = comb<KIND>(a1[w], v1[w]);
        }
        if (r < r1) {
            double v0[W];
            load_vec<DT_IN, W>(in, r * cols + col, v0);
#pragma unroll
            for (int w = 0; w < W; ++w) a0[w] = comb<KIND>(a0[w], v0[w]);
        }
    }
#pragma unroll
    for (int w = 0; w < W; ++w) smem[y][x * W + w] = comb<KIND>(a0[w], a1[w]);
    __syncthreads();
    // thread t of the first 32 * W finishes column bx * 32 * W + t
    for (uint32_t t = threadIdx.x; t < 32u * W; t += RT) {
        const uint64_t cc = (uint64_t)blockIdx.x * 32u * W + t;
        if (cc >= cols) continue;
        double v = smem[0][t];
#pragma unroll
        for (int k = 1; k < 8; ++k) v = comb<KIND>(v, smem[k][t]);
        store_from_double<DT_OUT>(dst, (uint64_t)blockIdx.y * cols + cc, v);
    }
}

// Whole-tensor reduction, one stage: CTA b reduces elements b * RT + t, stride gridDim.x * RT, to dst[b].
// W = 4 (n a multiple of 4, 16-byte aligned input): each thread reads four adjacent elements at a time; for sums the
// four are added pairwise in the input's widened binary32 first -- an error of at most 2^-24 of each small sum,
// whatever n is -- so that one conversion and one binary64 addition serve four elements.
template <int DT_IN, int DT_OUT, int KIND, int W>
__global__ void __launch_bounds__(RT) lt_reduce_all(const void *in, void *dst, uint64_t n) {
    __shared__ double smem[RT / 32];
    pdl_release();
    pdl_wait();
    const uint64_t stride = (uint64_t)gridDim.x * RT;
    double a0 = ident<KIND>(), a1 = ident<KIND>();
    if constexpr (W == 1) {
        uint64_t i = (uint64_t)blockIdx.x * RT + threadIdx.x;
        for (; i + stride < n; i += 2 * stride) {
            a0 = comb<KIND>(a0, load_as_double<DT_IN>(in, i));
            a1 = comb<KIND>(a1, load_as_double<DT_IN>(in, i + stride));
        }
        if (i < n) a0 = comb<KIND>(a0, load_as_double<DT_IN>(in, i));
    } else {
        auto fold = [](const double (&v)[W]) -> double {
            if constexpr (KIND == 0 && DT_IN != 5) return (double)(((float)v[0] + (float)v[1]) + ((float)v[2] + (float)v[3]));
            else return comb<KIND>(comb<KIND>(v[0], v[1]), comb<KIND>(v[2], v[3]));
        };
        const uint64_t nv = n / W;
        uint64_t i = (uint64_t)blockIdx.x * RT + threadIdx.x;
        for (; i + stride < nv; i += 2 * stride) {
            double v0[W], v1[W];
            load_vec<DT_IN, W>(in, i * W, v0);
            load_vec<DT_IN, W>(in, (i + stride) * W, v1);
            a0 = comb<KIND>(a0, fold(v0));
            a1 = comb<KIND>(a1, fold(v1));
        }
        if (i < nv) {
            double v0[W];
            load_vec<DT_IN, W>(in, i * W, v0);
            a0 = comb<KIND>(a0, fold(v0));
        }
    }
    const double v = cta_reduce<KIND>(comb<KIND>(a0, a1), smem);
    if (threadIdx.x == 0) store_from_double<DT_OUT>(dst, blockIdx.x, v);
}

template <int DT, int KIND>
cudaError_t launch_typed(int axis, const void *in, void *out, void *scratch, uint64_t rows, uint64_t cols, unsigned parts,
                         int sm_count, cudaStream_t stream, unsigned *launched) {
    constexpr int F64 = 5;
    if (axis == 0) {
        const unsigned grid = (unsigned)(rows < (uint64_t)sm_count * 8 ? (rows ? rows : 1) : (uint64_t)sm_count * 8);
        *launched = 1;
        return launch_pdl(lt_reduce_rows<DT, KIND>, grid, RT, (size_t)0, stream, in, out, (uint32_t)rows, cols);
    }
    if (axis == 1) {
        const bool wide = (cols % 4) == 0 && ((uintptr_t)in % 16) == 0;
        const unsigned gx = (unsigned)((cols + (wide ? 127 : 31)) / (wide ? 128 : 32));
        const unsigned gx2 = (unsigned)((cols + ((cols % 4) == 0 ? 127 : 31)) / ((cols % 4) == 0 ? 128 : 32));
        if (parts <= 1) {
            *launched = 1;
            return wide ? launch_pdl_grid(lt_reduce_cols<DT, DT, KIND, 4>, dim3(gx, 1), RT, stream, in, out, rows, cols, rows)
                        : launch_pdl_grid(lt_reduce_cols<DT, DT, KIND, 1>, dim3(gx, 1), RT, stream, in, out, rows, cols, rows);
        }
        const uint64_t rows_per = (rows + parts - 1) / parts;
        cudaError_t e = wide ? launch_pdl_grid(lt_reduce_cols<DT, F64, KIND, 4>, dim3(gx, parts), RT, stream, in, scratch, rows, cols, rows_per)
                             : launch_pdl_grid(lt_reduce_cols<DT, F64, KIND, 1>, dim3(gx, parts), RT, stream, in, scratch, rows, cols, rows_per);
        if (e != cudaSuccess) return e;
        *launched = 2;
        // the partial results: binary64, 256-byte aligned scratch
        return (cols % 4) == 0
                   ? launch_pdl_grid(lt_reduce_cols<F64, DT, KIND, 4>, dim3(gx2, 1), RT, stream, (const void *)scratch, out, (uint64_t)parts, cols, (uint64_t)parts)
                   : launch_pdl_grid(lt_reduce_cols<F64, DT, KIND, 1>, dim3(gx2, 1), RT, stream, (const void *)scratch, out, (uint64_t)parts, cols, (uint64_t)parts);
    }
    const uint64_t n = rows * cols;
    if (parts <= 1) {
        *launched = 1;
        return launch_pdl(lt_reduce_all<DT, DT, KIND, 1>, 1u, RT, (size_t)0, stream, in, out, n);
    }
    const bool wide = (n % 4) == 0 && ((uintptr_t)in % 16) == 0;
    cudaError_t e = wide ? launch_pdl(lt_reduce_all<DT, F64, KIND, 4>, parts, RT, (size_t)0, stream, in, scratch, n)
                         : launch_pdl(lt_reduce_all<DT, F64, KIND, 1>, parts, RT, (size_t)0, stream, in, scratch, n);
    if (e != cudaSuccess) return e;
    *launched = 2;
    return launch_pdl(lt_reduce_all<F64, DT, KIND, 1>, 1u, RT, (size_t)0, stream, (const void *)scratch, out, (uint64_t)parts);
}

template <int DT>
cudaError_t launch_kind(int axis, int kind, const void *in, void *out, void *scratch, uint64_t rows, uint64_t cols, unsigned parts,
                        int sm_count, cudaStream_t stream, unsigned *launched) {
    if (kind == 0) return launch_typed<DT, 0>(axis, in, out, scratch, rows, cols, parts, sm_count, stream, launched);
    if (kind == 1) return launch_typed<DT, 1>(axis, in, out, scratch, rows, cols, parts, sm_count, stream, launched);
    return launch_typed<DT, 2>(axis, in, out, scratch, rows, cols, parts, sm_count, stream, launched);
}

}  // namespace

unsigned lt_reduce_parts(int axis, uint64_t rows, uint64_t cols, int sm_count) {
    if (axis == 0) return 0;
    if (axis == 1) {
        // enough CTAs to fill the device a few times over, at least 64 rows each
        const uint64_t gx = (cols + 127) / 128;
        uint64_t want = ((uint64_t)sm_count * 8 + gx - 1) / gx;
        const uint64_t most = (rows + 63) / 64;
        if (want > most) want = most;
        if (want > 1024) want = 1024;
        return want < 1 ? 1u : (unsigned)want;
    }
    const uint64_t n = rows * cols;
    uint64_t want = (n + (uint64_t)RT * 16 - 1) / ((uint64_t)RT * 16);
    if (want > (uint64_t)sm_count * 8) want = (uint64_t)sm_count * 8;
    return want < 1 ? 1u : (unsigned)want;
}

size_t lt_reduce_scratch_bytes(int axis, uint64_t rows, uint64_t cols, int sm_count) {
    const unsigned parts = lt_reduce_parts(axis, rows, cols, sm_count);
    if (parts <= 1) return 0;
    return axis == 1 ? (size_t)parts * cols * sizeof(double) : (size_t)parts * sizeof(double);
}

namespace {
template <int DT, int KIND>
cudaError_t launch_final(int axis, const void *partials, void *out, unsigned parts, uint64_t cols, cudaStream_t stream) {
    constexpr int F64 = 5;
    if (axis == 1) {
        const unsigned gx = (unsigned)((cols + ((cols % 4) == 0 ? 127 : 31)) / ((cols % 4) == 0 ? 128 : 32));
        return (cols % 4) == 0 ? launch_pdl_grid(lt_reduce_cols<F64, DT, KIND, 4>, dim3(gx, 1), RT, stream, partials, out, (uint64_t)parts, cols, (uint64_t)parts)
                               : launch_pdl_grid(lt_reduce_cols<F64, DT, KIND, 1>, dim3(gx, 1), RT, stream, partials, out, (uint64_t)parts, cols, (uint64_t)parts);
    }
    return launch_pdl(lt_reduce_all<F64, DT, KIND, 1>, 1u, RT, (size_t)0, stream, partials, out, (uint64_t)parts);
}
}  // namespace

cudaError_t lt_launch_reduce_final(int axis, int kind, int dtype, const void *partials, void *out, unsigned parts, uint64_t cols, cudaStream_t stream) {
    if (dtype != 0 && dtype != 1) return cudaErrorInvalidValue;
#define LT_FINAL(DT)                                                                              \
    (kind == 0 ? launch_final<DT, 0>(axis, partials, out, parts, cols, stream)                    \
               : kind == 1 ? launch_final<DT, 1>(axis, partials, out, parts, cols, stream) : launch_final<DT, 2>(axis, partials, out, parts, cols, stream))
    return dtype == 0 ? LT_FINAL(0) : LT_FINAL(1);
#undef LT_FINAL
}

cudaError_t lt_launch_reduce(int axis, int kind, int dtype, const void *in, void *out, void *scratch, uint64_t rows, uint64_t cols,
                             int sm_count, cudaStream_t stream, unsigned *launched) {
    const unsigned parts = lt_reduce_parts(axis, rows, cols, sm_count);
    *launched = 0;
    if (dtype == 0) return launch_kind<0>(axis, kind, in, out, scratch, rows, cols, parts, sm_count, stream, launched);
    if (dtype == 1) return launch_kind<1>(axis, kind, in, out, scratch, rows, cols, parts, sm_count, stream, launched);
    return cudaErrorInvalidValue;
}
