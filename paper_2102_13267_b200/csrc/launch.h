// Host-callable launch wrappers of the three kernels (defined in kernels.cu).
// flavour: 0 fast (approximate transcendentals, for bf16 results), 1 precise (every op within 2 ulp),
// 2 ieee (division, square root and reciprocal correctly rounded as well).
#pragma once
#include <cuda_runtime_api.h>
#include <stddef.h>

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
