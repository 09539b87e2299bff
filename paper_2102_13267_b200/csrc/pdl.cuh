// Programmatic dependent launch, shared by the interpreter and the compiled shells.
//
// A kernel launched with the stream-serialisation attribute may begin (parameter reads, program staging, index
// arithmetic) while the kernel ahead of it on the stream is still draining.  pdl_wait() returns once that kernel
// has completed and its writes are visible; every global access of a kernel comes after it, so results do not
// depend on the overlap.  pdl_release() lets the next kernel on the stream be scheduled as soon as this one
// leaves room.  Without a kernel directly ahead on the stream both are no-ops.
#pragma once
#ifndef __CUDACC_RTC__
#include <cuda_runtime.h>

#include <utility>
#endif

#ifndef LT_PDL
#define LT_PDL 1
#endif

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

#ifndef __CUDACC_RTC__
template <class... KArgs, class... Args>
cudaError_t launch_pdl_grid(void (*kernel)(KArgs...), dim3 grid, unsigned threads, cudaStream_t stream, Args &&...args);

template <class... KArgs, class... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), unsigned grid, unsigned threads, size_t dyn, cudaStream_t stream, Args &&...args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = dyn;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = LT_PDL;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

template <class... KArgs, class... Args>
cudaError_t launch_pdl_grid(void (*kernel)(KArgs...), dim3 grid, unsigned threads, cudaStream_t stream, Args &&...args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = LT_PDL;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}
#endif  // !__CUDACC_RTC__
