// Host-callable launch wrappers of the three kernels (defined in kernels.cu).
#pragma once
#include <cuda_runtime_api.h>

#include "vm.h"



cudaError_t lt_launch_ew(const LtKParams &p, bool fast, unsigned grid, cudaStream_t stream);
cudaError_t lt_launch_row(const LtKParams &p, bool fast, unsigned grid, unsigned threads, cudaStream_t stream);
cudaError_t lt_launch_multi(const LtMultiParams &p, bool fast, unsigned grid, cudaStream_t stream);
cudaError_t lt_kernel_occupancy(int *ew_blocks_per_sm, int *row_blocks_per_sm_256, int *multi_blocks_per_sm);
