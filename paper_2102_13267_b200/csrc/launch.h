// Host-callable launch wrappers of the three kernels (defined in kernels.cu).
// flavour: 0 fast (approximate transcendentals, for bf16 results), 1 precise (every op within 2 ulp),
// 2 ieee (division, square root and reciprocal correctly rounded as well).
#pragma once
#include <cuda_runtime_api.h>
#include <stddef.h>
#include <stdint.h>

#include "vm.h"



cudaError_t lt_launch_ew(const LtKParams &p, int flavour, unsigned grid, cudaStream_t stream);
cudaError_t lt_launch_row(const LtKParams &p, int flavour, unsigned grid, unsigned threads, cudaStream_t stream);
cudaError_t lt_launch_multi(const LtMultiParams &p, int flavour, unsigned grid, cudaStream_t stream);
#ifndef LT_MAX_STAGE_BYTES
#define LT_MAX_STAGE_BYTES (64u * 1024u)
#endif  // staging buffers per thread block

// once per device: allow up to `max_stage_bytes` of dynamic shared memory for the staging buffers
cudaError_t lt_kernel_setup(size_t max_stage_bytes);
cudaError_t lt_kernel_occupancy(int *ew_blocks_per_sm, int *row_blocks_per_sm_256, int *multi_blocks_per_sm);

// static_scratch.cu: zero-fills `bytes` of the fixed scratch array at `base` on `stream`
cudaError_t lt_static_scratch_clear_enqueue(void *base, size_t bytes, int sm_count, cudaStream_t stream);

// reduce.cu: reductions that run as kernels of their own.  axis 0: rows of [rows, cols] -> out[rows]; 1: columns ->
// out[cols]; 2: everything -> out[1].  kind 0 sum, 1 max, 2 min; dtype 0 f32, 1 bf16 (input and result).
// The column and whole-tensor forms need lt_reduce_scratch_bytes of scratch memory (0 for small inputs).
// *launched receives the number of kernels enqueued (1 or 2).
size_t lt_reduce_scratch_bytes(int axis, uint64_t rows, uint64_t cols, int sm_count);
cudaError_t lt_launch_reduce(int axis, int kind, int dtype, const void *in, void *out, void *scratch, uint64_t rows, uint64_t cols,
                             int sm_count, cudaStream_t stream, unsigned *launched);
// How many partial results the first stage leaves per column (axis 1) or in all (axis 2); <= 1: one stage, no scratch.
unsigned lt_reduce_parts(int axis, uint64_t rows, uint64_t cols, int sm_count);
// The second stage alone: `parts` binary64 partial results per column (axis 1, partials[part * cols + col]) or in all
// (axis 2) -- what the first stage, or an elementwise kernel that reduces its result (lt_c_ewred), left in scratch.
cudaError_t lt_launch_reduce_final(int axis, int kind, int dtype, const void *partials, void *out, unsigned parts, uint64_t cols,
                                   cudaStream_t stream);

// views.cu: copy kernels of the shape operations.  `op` is the lt_opcode (reshape 60, narrow 61, permute 62,
// update_slice 63); in_dims is the (first) input's shape (reshape: {numel}), out_dims the result's (update_slice:
// the update's); a0 / a1 as recorded (dimension and start; packed permutation).  `in_place` non-zero: update_slice
// whose result already holds the base.  *launched receives the number of kernels enqueued.
cudaError_t lt_launch_view(int op, int elem_bytes, int rank, const int64_t *in_dims, const int64_t *out_dims, int64_t a0, int64_t a1,
                           const void *in, const void *upd, void *out, int in_place, int sm_count, cudaStream_t stream, unsigned *launched);
