// Table of ahead-of-time compiled programs (compiled.cu): lookup by exact program, launch by index.
#pragma once
#include <cuda_runtime_api.h>
#include <stdint.h>

#include "vm.h"

// Index of the table entry whose kernel family (0 elementwise, 1 row, 2 multi-tensor), flavour, instructions,
// prologue length and slot dtypes / classes equal the arguments, or -1.
int lt_compiled_find(int kind, int flavour, const LtIns *ins, uint32_t n_ins, uint32_t n_pro, const uint8_t *dtype,
                     const uint8_t *cls, uint32_t n_slots);
int lt_compiled_count(void);
const char *lt_compiled_name(int id);
// `u`: chunks of eight elements a thread keeps in flight (elementwise, multi: 1 or 2; row: 1, 2, 4 or 8).
// `params` points at the LtKParams (elementwise, row) or LtMultiParams block.  Row launches: `threads` per
// CTA and the power-of-two `group` of threads that owns a row.
// `depth`: row launches with 128-thread CTAs may keep the inputs of the next `depth` (1..4) blocks of rows in
// flight in shared memory (depth x lt_compiled_row_stage_bytes of dynamic shared memory); 0 = load directly.
cudaError_t lt_compiled_launch(int id, const void *params, int u, unsigned grid, unsigned threads, unsigned group,
                               unsigned group_log2, unsigned depth, cudaStream_t stream);
cudaError_t lt_compiled_occupancy(int id, int u, int threads, size_t dyn_smem, int *blocks_per_sm);
size_t lt_compiled_row_stage_bytes(int id, int u);
// 1 if the entry's row kernel gains from the staging ring, 0 for issue-bound programs (random-bit generation).
int lt_compiled_prefers_staging(int id);
// Accesses the compiled shells found outside their slots since the library was loaded (debug build with
// -DLT_DEBUG_BOUNDS only): 0 = *out is valid, 1 = not a debug build, -1 = the read failed.  Synchronises the device.
int lt_compiled_bounds_violations(unsigned long long *out);

// Long rows (more columns than a row's thread group keeps in registers): a CTA walks the row in slices, one pass
// per reduction plus one.  lt_compiled_long_stage_bytes: shared memory one staged row of the entry's full-class
// inputs takes at `cols` columns, 0 when they cannot be staged (a row that is not a multiple of 16 bytes).
// `depth` 0 = passes read global memory, 1 or 2 = rows staged that far ahead by bulk asynchronous copies whose
// completion the kernel awaits for at most `limit_ns` nanoseconds.
size_t lt_compiled_long_stage_bytes(int id, uint32_t cols);
// `threads`: 256 or 512 per CTA.  `l2_ahead` non-zero: the row a CTA takes next is requested into L2 while it works.
cudaError_t lt_compiled_launch_long(int id, const void *params, unsigned grid, unsigned threads, unsigned depth, size_t stage_bytes,
                                    uint64_t limit_ns, int l2_ahead, cudaStream_t stream);
cudaError_t lt_compiled_long_occupancy(int id, unsigned threads, size_t dyn_smem, int *blocks);
// Rows of up to 8 x 128 x 8 chunks whose thread group is a thread-block cluster of `cluster_size` (2, 4 or 8) CTAs of
// 128 threads, `u` (1, 2, 4 or 8) chunks per thread, the row in registers: `clusters` clusters share the rows.
// `depth` as for lt_compiled_launch (stages of lt_compiled_row_stage_bytes each); `limit_ns` bounds the wait of a
// reduction for the other CTAs' parts.  lt_compiled_cluster_occupancy: how many such clusters the device holds at once.
// `shared_vectors` non-zero: the program's column vectors (a thread's columns of gamma, beta, a bias) are kept in
// lt_compiled_cluster_vector_bytes of shared memory for the whole launch instead of being re-read for every row; zero:
// in registers when they fit 64 of them, else re-read.
cudaError_t lt_compiled_launch_cluster(int id, const void *params, int u, int shared_vectors, unsigned clusters, unsigned cluster_size,
                                       unsigned depth, uint64_t limit_ns, cudaStream_t stream);
cudaError_t lt_compiled_cluster_occupancy(int id, int u, int shared_vectors, unsigned cluster_size, unsigned depth, int *max_clusters);
size_t lt_compiled_cluster_vector_bytes(int id, int u);
// An elementwise entry whose result is reduced instead of stored (a slot of class LT_CLS_REDUCED...): the first stage,
// a grid of gx x gy CTAs of 256 threads.  Reduction over the rows of every column: gx = ceil(chunks per row / 32), CTA row
// `by` takes the rows [by * rows_per, ..) and writes cols binary64 partials at partial + by * cols.  Over everything:
// gy = 1 and gx partials.  The second stage is lt_launch_reduce_final (launch.h).
cudaError_t lt_compiled_launch_reduced(int id, const void *params, unsigned gx, unsigned gy, unsigned rows_per, cudaStream_t stream);
// Device status word (bit 0: a bounded wait gave up); synchronises the device.  `clear` resets it when set.
cudaError_t lt_device_status_read(unsigned int *out, int clear);
// Launches a one-warp kernel that waits `limit_ns` for an mbarrier phase nothing completes and then raises bit 0.
cudaError_t lt_wait_probe_launch(uint64_t limit_ns, cudaStream_t stream);
