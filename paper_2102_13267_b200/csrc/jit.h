// Run-time specialisation of the compiled shells for programs without a table entry (jit.cpp).
#pragma once
#include <stddef.h>
#include <stdint.h>

#include <atomic>
#include <map>
#include <memory>
#include <mutex>
#include <string>
#include <vector>

#include "vm.h"

namespace lt {

// Identity of a program as the shells see it, plus which instantiation its launches need.
struct JitProgram {
    int kind = 0;      // 0 elementwise, 1 row, 2 multi-tensor
    int flavour = 1;
    uint32_t n_pro = 0;
    std::vector<LtIns> ins;
    std::vector<uint8_t> dtype, cls;  // per slot
    bool long_row = false;            // row programs: the long-row shell (both CTA sizes) instead of lt_c_row
    int row_u = 1;                    // row programs: chunks per thread of the lt_c_row instantiation
    int cluster_u = 0;                // long rows: chunks per thread of the cluster row kernel (lt_c_rowc), 0 = not built
};

struct JitKernel {
    JitProgram program;
    std::atomic<int> state{0};  // 0 being compiled, 1 machine code ready, -1 failed (see log)
    std::string log;
    std::vector<char> cubin;
    std::string entry[4];       // lowered kernel names (long rows: 256- and 512-thread CTAs, cluster row kernel without / with column vectors in shared memory)
    struct Loaded {
        bool ok = false;
        void *fn[4] = {nullptr, nullptr, nullptr, nullptr};
    };
    std::mutex load_lock;
    std::map<int, Loaded> loaded;  // per device ordinal
};

bool jit_available();
// The kernel of `p`: from the process-wide cache, else compiled now (`synchronous`) or queued for the worker thread.
std::shared_ptr<JitKernel> jit_request(const JitProgram &p, bool synchronous);
bool jit_supported(const JitProgram &p);
// Loads the machine code on `device` (current on the calling thread) the first time; false if not ready or failed.
bool jit_load(JitKernel &k, int device, std::string *err);
int jit_occupancy(JitKernel &k, int device, int variant, int threads, size_t dyn_smem);
// `cluster` > 0: the grid is launched as thread-block clusters of that many CTAs.
bool jit_launch(JitKernel &k, int device, int variant, unsigned grid, unsigned threads, size_t dyn_smem, void *stream, void **args,
                std::string *err, unsigned cluster = 0, unsigned grid_y = 1);
// Clusters of `cluster` CTAs of `threads` threads the device holds at once (0: unknown or none).
int jit_cluster_occupancy(JitKernel &k, int device, int variant, int threads, unsigned cluster, size_t dyn_smem);
size_t jit_row_stage_bytes(const JitProgram &p, int u, int threads);
bool jit_integer_heavy(const JitProgram &p);
size_t jit_long_stage_bytes(const JitProgram &p, uint32_t cols);
int jit_reductions(const JitProgram &p);
// The slot an elementwise program reduces instead of storing (class LT_CLS_REDUCED...), or -1.
int jit_reduced_slot(const JitProgram &p);
// Shared memory the cluster row kernel needs to keep the program's column vectors at `u` chunks per thread (0: it has none).
size_t jit_cluster_vector_bytes(const JitProgram &p, int u);

}  // namespace lt
