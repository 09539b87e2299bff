// Ahead-of-time compiled programs.
//
// The planner's register programs (vm.h) are normally interpreted.  For the programs listed in
// compiled_programs.inc the same per-lane operations are instantiated at build time over the
// program itself: the instruction stream is a template parameter, every opcode test is resolved
// by the compiler, and what remains is the straight-line kernel one would write by hand for that
// fusion group -- no dispatch, no program fetch, registers allocated by ptxas.  The planner looks a
// group's program up in this table (exact match of instructions, slot dtypes and classes); a group
// that is not listed, or a launch whose pointers or extents do not allow 128-bit accesses, runs on
// the interpreter instead.  Immediates, pointers and extents stay run-time parameters, so one
// entry serves every shape and every value of the dynamic scalars.
//
// Three shells, as for the interpreter:
//   lt_c_ew     chunks of 8 elements strided over the grid, U chunks in flight per thread; many short CTAs
//               (a compiled CTA has no set-up to amortise)
//   lt_c_row    a power-of-two group of threads owns a row and keeps it in registers (U chunks of
//               8 elements per thread) across the row reductions; groups of up to 32 threads reduce
//               with shuffles alone, larger ones exchange warp partials through shared memory.
//               Persistent CTAs; the inputs of the next blocks of rows travel through a cp.async
//               staging ring (not for programs bound by integer issue), small column vectors are
//               loaded once per thread
//   lt_c_multi  one program over many tensors; a CTA takes super-chunks of 16384 elements and
//               finds the owning tensor by binary search over a prefix table in the parameters
// Every global access is a 128-bit (64-bit for one-byte types) access of a full chunk; full-class
// inputs are all requested at the top of an iteration, before any arithmetic or store.
#include <cuda_runtime.h>
#include <stdint.h>

#include "compiled.h"
#include "compiled_shells.cuh"

namespace {

// ------------------------------------------------------------------ table
#include "compiled_programs.inc"

template <class PG>
bool same_program(const LtIns *ins, uint32_t n_ins, uint32_t n_pro, const uint8_t *dtype, const uint8_t *cls, uint32_t n_slots) {
    if (n_ins != (uint32_t)PG::n_ins || n_pro != (uint32_t)PG::n_pro || n_slots != (uint32_t)PG::n_slots) return false;
    for (int i = 0; i < PG::n_ins; ++i)
        if (ins[i].op != PG::ins[i].op || ins[i].imm != PG::ins[i].imm) return false;
    for (int s = 0; s < PG::n_slots; ++s)
        if (dtype[s] != PG::dtype[s] || cls[s] != PG::cls[s]) return false;
    return true;
}

inline cudaError_t row_smem_attr(const void *kernel, size_t dyn) {
    // opt in to more than 48 KB of dynamic shared memory; per kernel, cheap enough to repeat per launch
    return dyn > 32u * 1024u ? cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) : cudaSuccess;
}


template <class PG, int U>
cudaError_t launch_row(const LtKParams &P, unsigned grid, unsigned threads, unsigned group, unsigned group_log2, unsigned depth,
                       cudaStream_t stream) {
    const size_t dyn = (size_t)depth * Info<PG>::stage_bytes(U, C_ROW_THREADS);
    cudaError_t e = row_smem_attr((const void *)lt_c_row<PG, U>, dyn);
    if (e != cudaSuccess) return e;
    return launch_pdl(lt_c_row<PG, U>, grid, threads, dyn, stream, P, (uint32_t)group, (uint32_t)group_log2, (uint32_t)depth);
}

template <class PG>
cudaError_t launch_one(const void *params, int u, unsigned grid, unsigned threads, unsigned group, unsigned group_log2,
                       unsigned depth, cudaStream_t stream) {
    if constexpr (PG::kind == 0 && Info<PG>::accum_slot() >= 0) {
        return cudaErrorInvalidValue;  // launched through lt_compiled_launch_reduced
    } else if constexpr (PG::kind == 0) {
        const LtKParams &P = *static_cast<const LtKParams *>(params);
        return u >= 2 ? launch_pdl(lt_c_ew<PG, 2>, grid, C_THREADS, 0, stream, P) : launch_pdl(lt_c_ew<PG, 1>, grid, C_THREADS, 0, stream, P);
    } else if constexpr (PG::kind == 1) {
        const LtKParams &P = *static_cast<const LtKParams *>(params);
        if (u >= 8) return launch_row<PG, 8>(P, grid, threads, group, group_log2, depth, stream);
        if (u >= 4) return launch_row<PG, 4>(P, grid, threads, group, group_log2, depth, stream);
        if (u >= 2) return launch_row<PG, 2>(P, grid, threads, group, group_log2, depth, stream);
        return launch_row<PG, 1>(P, grid, threads, group, group_log2, depth, stream);
    } else {
        const LtMultiParams &P = *static_cast<const LtMultiParams *>(params);
        return u >= 2 ? launch_pdl(lt_c_multi<PG, 2>, grid, C_THREADS, 0, stream, P) : launch_pdl(lt_c_multi<PG, 1>, grid, C_THREADS, 0, stream, P);
    }
}

template <class PG, int U>
cudaError_t row_occupancy(int threads, size_t dyn, int *blocks) {
    cudaError_t e = row_smem_attr((const void *)lt_c_row<PG, U>, dyn);
    if (e != cudaSuccess) return e;
    return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks, lt_c_row<PG, U>, threads, dyn);
}

template <class PG>
cudaError_t occupancy_one(int u, int threads, size_t dyn, int *blocks) {
    if constexpr (PG::kind == 0 && Info<PG>::accum_slot() >= 0) {
        return cudaErrorInvalidValue;
    } else if constexpr (PG::kind == 0) {
        return u >= 2 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks, lt_c_ew<PG, 2>, C_THREADS, 0)
                      : cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks, lt_c_ew<PG, 1>, C_THREADS, 0);
    } else if constexpr (PG::kind == 1) {
        if (u >= 8) return row_occupancy<PG, 8>(threads, dyn, blocks);
        if (u >= 4) return row_occupancy<PG, 4>(threads, dyn, blocks);
        if (u >= 2) return row_occupancy<PG, 2>(threads, dyn, blocks);
        return row_occupancy<PG, 1>(threads, dyn, blocks);
    } else {
        return u >= 2 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks, lt_c_multi<PG, 2>, C_THREADS, 0)
                      : cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks, lt_c_multi<PG, 1>, C_THREADS, 0);
    }
}

}  // namespace

int lt_compiled_find(int kind, int flavour, const LtIns *ins, uint32_t n_ins, uint32_t n_pro, const uint8_t *dtype,
                     const uint8_t *cls, uint32_t n_slots) {
    int id = 0;
#define LT_X(PG)                                                                                                  \
    if (PG::kind == kind && PG::flavour == flavour && same_program<PG>(ins, n_ins, n_pro, dtype, cls, n_slots)) return id; \
    ++id;
    LT_COMPILED_LIST(LT_X)
#undef LT_X
    return -1;
}

namespace {

template <class PG, int S = 0>
size_t long_stage_bytes(uint32_t cols) {
    if constexpr (S < PG::n_slots) {
        constexpr bool in = Info<PG>::full_input(S);
        constexpr int eb = Info<PG>::elem_bytes(S);
        return (in ? (((size_t)cols * eb + 15u) & ~(size_t)15u) : 0) + long_stage_bytes<PG, S + 1>(cols);
    } else {
        return 0;
    }
}

template <class PG, int S = 0>
bool long_stage_allowed(uint32_t cols) {  // every staged row a multiple of 16 bytes
    if constexpr (S < PG::n_slots) {
        constexpr bool in = Info<PG>::full_input(S);
        constexpr int eb = Info<PG>::elem_bytes(S);
        return !(in && ((size_t)cols * eb) % 16u) && long_stage_allowed<PG, S + 1>(cols);
    } else {
        return true;
    }
}

template <class PG, int T>
cudaError_t launch_long_t(const LtKParams &P, unsigned grid, unsigned depth, size_t stage_bytes, uint64_t limit_ns, bool l2_ahead,
                          cudaStream_t stream) {
    const size_t dyn = (size_t)depth * stage_bytes;
    cudaError_t e = row_smem_attr((const void *)lt_c_longrow<PG, T>, dyn);
    if (e != cudaSuccess) return e;
    return launch_pdl(lt_c_longrow<PG, T>, grid, (unsigned)T, dyn, stream, P, (uint32_t)depth, (uint32_t)stage_bytes, limit_ns,
                      (uint32_t)(l2_ahead ? 1 : 0));
}

template <class PG>
cudaError_t launch_long(const LtKParams &P, unsigned grid, unsigned threads, unsigned depth, size_t stage_bytes, uint64_t limit_ns,
                        bool l2_ahead, cudaStream_t stream) {
    if constexpr (PG::kind == 1 && Info<PG>::n_reds() <= 4) {
        return threads >= 512 ? launch_long_t<PG, 512>(P, grid, depth, stage_bytes, limit_ns, l2_ahead, stream)
                              : launch_long_t<PG, 256>(P, grid, depth, stage_bytes, limit_ns, l2_ahead, stream);
    } else {
        return cudaErrorInvalidValue;
    }
}

template <class PG>
cudaError_t long_occupancy(unsigned threads, size_t dyn, int *blocks) {
    if constexpr (PG::kind == 1 && Info<PG>::n_reds() <= 4) {
        if (threads >= 512) {
            cudaError_t e = row_smem_attr((const void *)lt_c_longrow<PG, 512>, dyn);
            if (e != cudaSuccess) return e;
            return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks, lt_c_longrow<PG, 512>, 512, dyn);
        }
        cudaError_t e = row_smem_attr((const void *)lt_c_longrow<PG, 256>, dyn);
        if (e != cudaSuccess) return e;
        return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks, lt_c_longrow<PG, 256>, 256, dyn);
    } else {
        return cudaErrorInvalidValue;
    }
}

// Cluster row kernel: launched with the cluster dimension and the programmatic-launch attribute; with no parameter
// block, answers how many clusters the device holds at once instead
template <class PG, int U, bool HS>
cudaError_t rowc_do(const LtKParams *P, unsigned clusters, unsigned cluster_size, unsigned depth, uint64_t limit_ns, cudaStream_t stream,
                    int *max_clusters) {
    const size_t dyn = (size_t)depth * Info<PG>::stage_bytes(U, C_ROW_THREADS) + (HS ? (size_t)Info<PG>::n_reserved() * U * C_ROW_THREADS * 32u : 0u);
    cudaError_t e = row_smem_attr((const void *)lt_c_rowc<PG, U, HS>, dyn);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((clusters ? clusters : 1u) * cluster_size);
    cfg.blockDim = dim3(C_ROW_THREADS);
    cfg.dynamicSmemBytes = dyn;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster_size;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = LT_PDL;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (!P) {
        cfg.numAttrs = 1;  // the occupancy query takes the cluster dimension only
        return cudaOccupancyMaxActiveClusters(max_clusters, lt_c_rowc<PG, U, HS>, &cfg);
    }
    return cudaLaunchKernelEx(&cfg, lt_c_rowc<PG, U, HS>, *P, (uint32_t)depth, limit_ns);
}

// `shared_vectors`: column vectors of the program kept in shared memory (only instantiated for programs that have some)
template <class PG>
cudaError_t rowc_one(const LtKParams *P, int u, bool shared_vectors, unsigned clusters, unsigned cluster_size, unsigned depth, uint64_t limit_ns,
                     cudaStream_t stream, int *max_clusters) {
    if constexpr (PG::kind == 1) {
        if constexpr (Info<PG>::n_reserved() > 0) {
            if (shared_vectors) {
                if (u >= 8) return rowc_do<PG, 8, true>(P, clusters, cluster_size, depth, limit_ns, stream, max_clusters);
                if (u >= 4) return rowc_do<PG, 4, true>(P, clusters, cluster_size, depth, limit_ns, stream, max_clusters);
                if (u >= 2) return rowc_do<PG, 2, true>(P, clusters, cluster_size, depth, limit_ns, stream, max_clusters);
                return rowc_do<PG, 1, true>(P, clusters, cluster_size, depth, limit_ns, stream, max_clusters);
            }
        }
        if (u >= 8) return rowc_do<PG, 8, false>(P, clusters, cluster_size, depth, limit_ns, stream, max_clusters);
        if (u >= 4) return rowc_do<PG, 4, false>(P, clusters, cluster_size, depth, limit_ns, stream, max_clusters);
        if (u >= 2) return rowc_do<PG, 2, false>(P, clusters, cluster_size, depth, limit_ns, stream, max_clusters);
        return rowc_do<PG, 1, false>(P, clusters, cluster_size, depth, limit_ns, stream, max_clusters);
    } else {
        return cudaErrorInvalidValue;
    }
}

}  // namespace

namespace {
template <class PG>
cudaError_t launch_reduced(const LtKParams &P, unsigned gx, unsigned gy, unsigned rows_per, cudaStream_t stream) {
    if constexpr (PG::kind == 0 && Info<PG>::accum_slot() >= 0) {
        return launch_pdl_grid(lt_c_ewred<PG>, dim3(gx, gy), (unsigned)C_THREADS, stream, P, (uint32_t)rows_per);
    } else {
        return cudaErrorInvalidValue;
    }
}
}  // namespace

cudaError_t lt_compiled_launch_reduced(int id, const void *params, unsigned gx, unsigned gy, unsigned rows_per, cudaStream_t stream) {
    int k = 0;
#define LT_X(PG)                                                                                            \
    if (k == id) return launch_reduced<PG>(*static_cast<const LtKParams *>(params), gx, gy, rows_per, stream); \
    ++k;
    LT_COMPILED_LIST(LT_X)
#undef LT_X
    return cudaErrorInvalidValue;
}

size_t lt_compiled_cluster_vector_bytes(int id, int u) {
    int k = 0;
#define LT_X(PG)                                                                          \
    if (k == id) return (size_t)Info<PG>::n_reserved() * (size_t)u * C_ROW_THREADS * 32u; \
    ++k;
    LT_COMPILED_LIST(LT_X)
#undef LT_X
    return 0;
}

cudaError_t lt_compiled_launch_cluster(int id, const void *params, int u, int shared_vectors, unsigned clusters, unsigned cluster_size,
                                       unsigned depth, uint64_t limit_ns, cudaStream_t stream) {
    int k = 0;
#define LT_X(PG)                                                                                                                        \
    if (k == id) return rowc_one<PG>(static_cast<const LtKParams *>(params), u, shared_vectors != 0, clusters, cluster_size, depth, limit_ns, stream, nullptr); \
    ++k;
    LT_COMPILED_LIST(LT_X)
#undef LT_X
    return cudaErrorInvalidValue;
}

cudaError_t lt_compiled_cluster_occupancy(int id, int u, int shared_vectors, unsigned cluster_size, unsigned depth, int *max_clusters) {
    int k = 0;
#define LT_X(PG)                                                                                  \
    if (k == id) return rowc_one<PG>(nullptr, u, shared_vectors != 0, 0, cluster_size, depth, 0, nullptr, max_clusters); \
    ++k;
    LT_COMPILED_LIST(LT_X)
#undef LT_X
    return cudaErrorInvalidValue;
}

size_t lt_compiled_long_stage_bytes(int id, uint32_t cols) {
    int k = 0;
#define LT_X(PG)                                                                  \
    if (k == id) return long_stage_allowed<PG>(cols) ? long_stage_bytes<PG>(cols) : 0; \
    ++k;
    LT_COMPILED_LIST(LT_X)
#undef LT_X
    return 0;
}

cudaError_t lt_compiled_launch_long(int id, const void *params, unsigned grid, unsigned threads, unsigned depth, size_t stage_bytes,
                                    uint64_t limit_ns, int l2_ahead, cudaStream_t stream) {
    int k = 0;
#define LT_X(PG)                                                                                                                  \
    if (k == id)                                                                                                                  \
        return launch_long<PG>(*static_cast<const LtKParams *>(params), grid, threads, depth, stage_bytes, limit_ns, l2_ahead != 0, stream); \
    ++k;
    LT_COMPILED_LIST(LT_X)
#undef LT_X
    return cudaErrorInvalidValue;
}

cudaError_t lt_compiled_long_occupancy(int id, unsigned threads, size_t dyn_smem, int *blocks) {
    int k = 0;
#define LT_X(PG)                                                  \
    if (k == id) return long_occupancy<PG>(threads, dyn_smem, blocks); \
    ++k;
    LT_COMPILED_LIST(LT_X)
#undef LT_X
    return cudaErrorInvalidValue;
}

cudaError_t lt_device_status_read(unsigned int *out, int clear) {
    cudaError_t e = cudaMemcpyFromSymbol(out, lt_device_status, sizeof(*out));
    if (e == cudaSuccess && clear && *out) {
        const unsigned int zero = 0;
        e = cudaMemcpyToSymbol(lt_device_status, &zero, sizeof(zero));
    }
    return e;
}

cudaError_t lt_wait_probe_launch(uint64_t limit_ns, cudaStream_t stream) {
    lt_wait_probe<<<1, 32, 0, stream>>>(limit_ns);
    return cudaGetLastError();
}

int lt_compiled_bounds_violations(unsigned long long *out) {
#ifdef LT_DEBUG_BOUNDS
    return cudaMemcpyFromSymbol(out, lt_c_bounds_violations, sizeof(*out)) == cudaSuccess ? 0 : -1;
#else
    (void)out;
    return 1;  // not a debug build
#endif
}

int lt_compiled_count(void) {
    int n = 0;
#define LT_X(PG) ++n;
    LT_COMPILED_LIST(LT_X)
#undef LT_X
    return n;
}

size_t lt_compiled_row_stage_bytes(int id, int u) {
    int k = 0;
#define LT_X(PG)                                                                                                        \
    if (k == id)                                                                                                        \
        return (size_t)(u >= 8 ? Info<PG>::stage_bytes(8, C_ROW_THREADS) : u >= 4 ? Info<PG>::stage_bytes(4, C_ROW_THREADS) \
                        : u >= 2 ? Info<PG>::stage_bytes(2, C_ROW_THREADS) : Info<PG>::stage_bytes(1, C_ROW_THREADS)); \
    ++k;
    LT_COMPILED_LIST(LT_X)
#undef LT_X
    return 0;
}

int lt_compiled_prefers_staging(int id) {
    int k = 0;
#define LT_X(PG)                                            \
    if (k == id) return Info<PG>::integer_heavy() ? 0 : 1; \
    ++k;
    LT_COMPILED_LIST(LT_X)
#undef LT_X
    return 0;
}

const char *lt_compiled_name(int id) {
    int k = 0;
#define LT_X(PG)                 \
    if (k == id) return PG::name; \
    ++k;
    LT_COMPILED_LIST(LT_X)
#undef LT_X
    return "";
}

cudaError_t lt_compiled_launch(int id, const void *params, int u, unsigned grid, unsigned threads, unsigned group,
                               unsigned group_log2, unsigned depth, cudaStream_t stream) {
    int k = 0;
#define LT_X(PG)                                                                                \
    if (k == id) return launch_one<PG>(params, u, grid, threads, group, group_log2, depth, stream); \
    ++k;
    LT_COMPILED_LIST(LT_X)
#undef LT_X
    return cudaErrorInvalidValue;
}

cudaError_t lt_compiled_occupancy(int id, int u, int threads, size_t dyn_smem, int *blocks) {
    int k = 0;
#define LT_X(PG)                                                  \
    if (k == id) return occupancy_one<PG>(u, threads, dyn_smem, blocks); \
    ++k;
    LT_COMPILED_LIST(LT_X)
#undef LT_X
    return cudaErrorInvalidValue;
}
