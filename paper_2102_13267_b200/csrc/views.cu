// Copy kernels behind the shape operations (reshape, narrow, permute, update_slice) when they are not folded
// into a program: every one reads dense row-major buffers and writes a dense row-major result.
//
// narrow and update_slice move a block of `rows` runs of `width` bytes between two pitches: seen as
// [A, L, B] (A = product of the dimensions before `dim`, L = its extent, B = product of those after), the slice
// [start, start + len) of every one of the A outer indices is one contiguous run of len * B elements.
// permute gathers: thread i of the result reads the source element its coordinates map to.
#include <cuda_runtime.h>
#include <stdint.h>

#include "launch.h"
#include "pdl.cuh"

namespace {

constexpr int VT = 256;

// rows x width bytes, in units of sizeof(T); src / dst advance by their pitch (in units) per row
template <class T>
__global__ void __launch_bounds__(VT) lt_copy_pitched(const T *__restrict__ src, T *__restrict__ dst, uint64_t rows, uint64_t width,
                                                      uint64_t src_pitch, uint64_t dst_pitch) {
    pdl_release();
    pdl_wait();
    const uint64_t total = rows * width;
    for (uint64_t i = (uint64_t)blockIdx.x * VT + threadIdx.x; i < total; i += (uint64_t)gridDim.x * VT) {
        const uint64_t r = i / width, x = i - r * width;
        dst[r * dst_pitch + x] = src[r * src_pitch + x];
    }
}

struct PermuteArgs {
    int rank;
    uint64_t out_dims[6];
    uint64_t src_stride[6];  // stride in the source of the dimension result dimension k runs over
};

template <class T>
__global__ void __launch_bounds__(VT) lt_permute_copy(const T *__restrict__ src, T *__restrict__ dst, uint64_t total, const PermuteArgs a) {
    pdl_release();
    pdl_wait();
    for (uint64_t i = (uint64_t)blockIdx.x * VT + threadIdx.x; i < total; i += (uint64_t)gridDim.x * VT) {
        uint64_t rest = i, off = 0;
#pragma unroll
        for (int k = 5; k >= 0; --k) {
            if (k >= a.rank) continue;
            const uint64_t q = rest / a.out_dims[k];
            off += (rest - q * a.out_dims[k]) * a.src_stride[k];
            rest = q;
        }
        dst[i] = src[off];
    }
}

unsigned grid_for(uint64_t items, int sm_count) {
    uint64_t g = (items + VT - 1) / VT;
    const uint64_t most = (uint64_t)sm_count * 16;
    if (g > most) g = most;
    return g < 1 ? 1u : (unsigned)g;
}

// largest unit of 16, 8, 4, 2 or 1 bytes that divides every address, pitch and width
int common_unit(uint64_t a, uint64_t b, uint64_t c, uint64_t d, uint64_t e) {
    const uint64_t all = a | b | c | d | e;
    for (int u = 16; u > 1; u >>= 1)
        if ((all & (uint64_t)(u - 1)) == 0) return u;
    return 1;
}

cudaError_t copy_pitched(const void *src, void *dst, uint64_t rows, uint64_t width_bytes, uint64_t src_pitch_bytes, uint64_t dst_pitch_bytes,
                         int sm_count, cudaStream_t stream) {
    if (rows == 0 || width_bytes == 0) return cudaSuccess;
    const int u = common_unit((uint64_t)(uintptr_t)src, (uint64_t)(uintptr_t)dst, width_bytes, src_pitch_bytes, dst_pitch_bytes);
    const uint64_t w = width_bytes / u, sp = src_pitch_bytes / u, dp = dst_pitch_bytes / u;
    const unsigned grid = grid_for(rows * w, sm_count);
    switch (u) {
    case 16: return launch_pdl(lt_copy_pitched<uint4>, grid, VT, (size_t)0, stream, (const uint4 *)src, (uint4 *)dst, rows, w, sp, dp);
    case 8: return launch_pdl(lt_copy_pitched<uint2>, grid, VT, (size_t)0, stream, (const uint2 *)src, (uint2 *)dst, rows, w, sp, dp);
    case 4: return launch_pdl(lt_copy_pitched<uint32_t>, grid, VT, (size_t)0, stream, (const uint32_t *)src, (uint32_t *)dst, rows, w, sp, dp);
    case 2: return launch_pdl(lt_copy_pitched<uint16_t>, grid, VT, (size_t)0, stream, (const uint16_t *)src, (uint16_t *)dst, rows, w, sp, dp);
    default: return launch_pdl(lt_copy_pitched<uint8_t>, grid, VT, (size_t)0, stream, (const uint8_t *)src, (uint8_t *)dst, rows, w, sp, dp);
    }
}

}  // namespace

cudaError_t lt_launch_view(int op, int elem_bytes, int rank, const int64_t *in_dims, const int64_t *out_dims, int64_t a0, int64_t a1,
                           const void *in, const void *upd, void *out, int in_place, int sm_count, cudaStream_t stream, unsigned *launched) {
    *launched = 1;
    const uint64_t es = (uint64_t)elem_bytes;
    if (op == 60) {  // reshape: the same bytes
        const uint64_t bytes = (uint64_t)in_dims[0] * es;
        return copy_pitched(in, out, 1, bytes, bytes, bytes, sm_count, stream);
    }
    if (op == 61 || op == 63) {  // narrow / update_slice along dimension a0 at a1; out_dims = the slice's shape
        uint64_t A = 1, B = 1;
        for (int d = 0; d < a0; ++d) A *= (uint64_t)in_dims[d];
        for (int d = (int)a0 + 1; d < rank; ++d) B *= (uint64_t)in_dims[d];
        const uint64_t L = (uint64_t)in_dims[a0], len = (uint64_t)out_dims[a0];
        const uint64_t run = len * B * es, full = L * B * es, off = (uint64_t)a1 * B * es;
        if (op == 61) return copy_pitched((const char *)in + off, out, A, run, full, run, sm_count, stream);
        if (!in_place) {
            cudaError_t e = copy_pitched(in, out, 1, A * full, A * full, A * full, sm_count, stream);
            if (e != cudaSuccess) return e;
            *launched = 2;
        }
        return copy_pitched(upd, (char *)out + off, A, run, run, full, sm_count, stream);
    }
    if (op == 62) {  // permute: result dimension k is source dimension (a0 >> 4k) & 15
        PermuteArgs a{};
        a.rank = rank;
        uint64_t stride[6] = {0}, s = 1, total = 1;
        for (int d = rank - 1; d >= 0; --d) {
            stride[d] = s;
            s *= (uint64_t)in_dims[d];
        }
        for (int k = 0; k < rank; ++k) {
            a.out_dims[k] = (uint64_t)out_dims[k];
            a.src_stride[k] = stride[(a0 >> (4 * k)) & 0xf];
            total *= a.out_dims[k];
        }
        if (total == 0) return cudaSuccess;
        const unsigned grid = grid_for(total, sm_count);
        if (es == 4) return launch_pdl(lt_permute_copy<uint32_t>, grid, VT, (size_t)0, stream, (const uint32_t *)in, (uint32_t *)out, total, a);
        if (es == 2) return launch_pdl(lt_permute_copy<uint16_t>, grid, VT, (size_t)0, stream, (const uint16_t *)in, (uint16_t *)out, total, a);
        return launch_pdl(lt_permute_copy<uint8_t>, grid, VT, (size_t)0, stream, (const uint8_t *)in, (uint8_t *)out, total, a);
    }
    return cudaErrorInvalidValue;
}
