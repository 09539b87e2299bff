// lt_barrier_static_scratch: a barrier for callers that cannot obtain device memory while
// they run -- control loops with a latency budget that has no room for an allocator call (which
// may synchronise the device), plug-ins that were handed a fixed carve-out of a GPU whose
// remaining memory belongs to the host application, processes started after another framework
// has already claimed the device's memory.  The kernels launched are the same ones lt_barrier
// launches; only the placement of the values that pass between two kernels of one flush differs:
// they live in the array below instead of memory taken from the context's allocator.
#include <cuda_runtime.h>

#include <mutex>
#include <string>

#include "engine.h"

#ifndef LT_STATIC_SCRATCH_BYTES
#define LT_STATIC_SCRATCH_BYTES (32u << 20)  // keep equal to the figure documented in lazytensor.h
#endif
static_assert(LT_STATIC_SCRATCH_BYTES == LT_STATIC_SCRATCH_MAX_BYTES, "header and array disagree");

// One copy per GPU that loads the library, held until the process exits.  In host code this name
// is only a handle for cudaGetSymbolAddress; kernels get the address that call returns.
static __device__ __align__(256) unsigned char lt_static_scratch[LT_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_setup_lock;
void *g_scratch_addr[kMaxDevices];  // per device ordinal, filled on first use

// Writes zeros over `n` 16-byte words starting at `p` (the array's device address on the launching device).
__global__ void lt_static_scratch_clear(uint4 *p, size_t n) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        p[i] = make_uint4(0u, 0u, 0u, 0u);
}

// Device address of the array on `device`, looked up once per device with that device current.
cudaError_t scratch_address(int device, void **out) {
    if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> hold(g_setup_lock);
    if (!g_scratch_addr[device]) {
        int previous = -1;
        cudaError_t e = cudaGetDevice(&previous);
        if (e == cudaSuccess && previous != device) e = cudaSetDevice(device);
        void *p = nullptr;
        if (e == cudaSuccess) e = cudaGetSymbolAddress(&p, lt_static_scratch);
        if (previous >= 0 && previous != device) cudaSetDevice(previous);
        if (e != cudaSuccess) return e;
        g_scratch_addr[device] = p;
    }
    *out = g_scratch_addr[device];
    return cudaSuccess;
}

// Restores what the call changed on the context, whichever way the call ends.
struct StaticModeScope {
    lt_ctx *c;
    StaticModeScope(lt_ctx *ctx, void *base) : c(ctx) {
        c->static_base = base;
        c->static_cap = LT_STATIC_SCRATCH_BYTES;
        c->static_mode = true;
    }
    ~StaticModeScope() {
        c->static_mode = false;
        c->static_clear = false;
    }
};

}  // namespace

// Called by the executor once a flush in static mode has passed its checks (every result has a caller
// buffer, the temporaries fit), just before the first kernel: a refused call leaves the array untouched.
cudaError_t lt_static_scratch_clear_enqueue(void *base, size_t bytes, int sm_count, cudaStream_t stream) {
    lt_static_scratch_clear<<<sm_count > 0 ? sm_count : 1, 256, 0, stream>>>(reinterpret_cast<uint4 *>(base), bytes / 16u);
    return cudaGetLastError();
}

extern "C" __attribute__((visibility("default"))) lt_status lt_barrier_static_scratch(lt_ctx *c, int blocking,
                                                                                      int clear_first) {
    if (!c) return LT_ERR_INVALID_ARG;
    if (c->device == LT_DEVICE_NONE)
        return lt::fail(c, LT_ERR_DEVICE, "lt_barrier_static_scratch needs a context on a CUDA device");
    void *base = nullptr;
    cudaError_t e = scratch_address(c->device, &base);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return lt::fail(c, LT_ERR_CUDA, std::string("cudaGetSymbolAddress(static scratch): ") + cudaGetErrorString(e));
    }
    // The array still holds what the previous flush left there.  No kernel of this library reads a
    // temporary before writing it, so clearing is only for callers that want a known state; the executor
    // enqueues it after the graph has passed the checks of this mode.
    lt::DeviceScope on_device(c->device);
    if (!on_device.ok()) return lt::fail(c, LT_ERR_CUDA, "cudaSetDevice failed for the context's device");
    StaticModeScope mode(c, base);
    c->static_clear = clear_first != 0;
    return lt_barrier(c, blocking);
}
