// Run-time specialisation: the kernels of compiled_shells.cuh, built for a program that has no entry in the
// build-time table.
//
// The paper's runtime compiles a traced graph once and caches the executable (Section 4).  This library normally
// needs no compiler at run time -- programs in the table have kernels, everything else is interpreted -- but a graph
// that keeps coming back deserves the straight-line kernel too.  For such a program the same hand-written shells
// are instantiated over the program by the CUDA run-time compiler (NVRTC, loaded with dlopen; if it or the driver
// library cannot be loaded the feature is simply absent), on a worker thread, while the interpreter keeps
// serving the flushes; once the machine code is there the launches switch over.  Nothing is generated but the
// program's table entry (a struct of constants): the kernels are the ones in compiled_shells.cuh.
#include "jit.h"

#include <cuda.h>
#include <dlfcn.h>
#include <nvrtc.h>

#include <condition_variable>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <deque>
#include <map>
#include <mutex>
#include <string>
#include <thread>
#include <vector>

namespace lt {

namespace {

#include "jit_sources.inc"  // the text of vm.h, vm_ops.cuh, pdl.cuh and compiled_shells.cuh

struct Api {
    bool ok = false;
    int compiler_version = 0;  // major * 1000 + minor * 10
    // NVRTC
    nvrtcResult (*CreateProgram)(nvrtcProgram *, const char *, const char *, int, const char *const *, const char *const *) = nullptr;
    nvrtcResult (*DestroyProgram)(nvrtcProgram *) = nullptr;
    nvrtcResult (*CompileProgram)(nvrtcProgram, int, const char *const *) = nullptr;
    nvrtcResult (*AddNameExpression)(nvrtcProgram, const char *) = nullptr;
    nvrtcResult (*GetLoweredName)(nvrtcProgram, const char *, const char **) = nullptr;
    nvrtcResult (*GetCUBINSize)(nvrtcProgram, size_t *) = nullptr;
    nvrtcResult (*GetCUBIN)(nvrtcProgram, char *) = nullptr;
    nvrtcResult (*GetProgramLogSize)(nvrtcProgram, size_t *) = nullptr;
    nvrtcResult (*GetProgramLog)(nvrtcProgram, char *) = nullptr;
    // driver
    CUresult (*ModuleLoadData)(CUmodule *, const void *) = nullptr;
    CUresult (*ModuleGetFunction)(CUfunction *, CUmodule, const char *) = nullptr;
    CUresult (*LaunchKernelEx)(const CUlaunchConfig *, CUfunction, void **, void **) = nullptr;
    CUresult (*FuncSetAttribute)(CUfunction, CUfunction_attribute, int) = nullptr;
    CUresult (*OccupancyMaxActiveBlocksPerMultiprocessor)(int *, CUfunction, int, size_t) = nullptr;
    CUresult (*GetErrorString)(CUresult, const char **) = nullptr;
    CUresult (*OccupancyMaxActiveClusters)(int *, CUfunction, const CUlaunchConfig *) = nullptr;
};

template <class F>
bool sym(void *lib, const char *name, F &fn) {
    fn = reinterpret_cast<F>(dlsym(lib, name));
    return fn != nullptr;
}

const Api &api() {
    static Api a = [] {
        Api x;
        void *drv = nullptr;
        for (const char *n : {"libcuda.so.1", "libcuda.so"})
            if (!drv) drv = dlopen(n, RTLD_NOW | RTLD_LOCAL);
        int driver_version = 0;  // e.g. 12090; 0 = unknown (no driver here: anything may compile, nothing is loaded)
        CUresult (*driver_get_version)(int *) = nullptr;
        if (drv && sym(drv, "cuDriverGetVersion", driver_get_version)) driver_get_version(&driver_version);
        // Several copies of the compiler can be installed (a toolkit's, and one bundled with a Python package that is
        // already mapped under the same soname, which a bare name would resolve to).  Their register allocation
        // differs measurably, so take the newest one the driver can load code from: LT_NVRTC names a file outright,
        // else the toolkit directories are tried by path before the bare names.
        std::vector<std::string> candidates;
        if (const char *e = getenv("LT_NVRTC")) candidates.push_back(e);
        else {
            for (const char *var : {"CUDA_HOME", "CUDA_PATH"})
                if (const char *e = getenv(var)) candidates.push_back(std::string(e) + "/lib64/libnvrtc.so.12");
            candidates.push_back("/usr/local/cuda/lib64/libnvrtc.so.12");
            candidates.push_back("libnvrtc.so.12");
            candidates.push_back("libnvrtc.so");
        }
        void *rtc = nullptr;
        int best = -1;
        for (const std::string &n : candidates) {
            void *h = dlopen(n.c_str(), RTLD_NOW | RTLD_LOCAL);
            if (!h) continue;
            nvrtcResult (*version)(int *, int *) = nullptr;
            int major = 0, minor = 0;
            const bool known = sym(h, "nvrtcVersion", version) && version(&major, &minor) == NVRTC_SUCCESS;
            const int v = known ? major * 1000 + minor * 10 : 0;
            if (v > best && (driver_version == 0 || v <= driver_version)) {
                if (rtc) dlclose(rtc);
                rtc = h, best = v;
            } else dlclose(h);
        }
        if (!rtc) return x;
        x.compiler_version = best;
        bool ok = sym(rtc, "nvrtcCreateProgram", x.CreateProgram) && sym(rtc, "nvrtcDestroyProgram", x.DestroyProgram) &&
                  sym(rtc, "nvrtcCompileProgram", x.CompileProgram) && sym(rtc, "nvrtcAddNameExpression", x.AddNameExpression) &&
                  sym(rtc, "nvrtcGetLoweredName", x.GetLoweredName) && sym(rtc, "nvrtcGetCUBINSize", x.GetCUBINSize) &&
                  sym(rtc, "nvrtcGetCUBIN", x.GetCUBIN) && sym(rtc, "nvrtcGetProgramLogSize", x.GetProgramLogSize) &&
                  sym(rtc, "nvrtcGetProgramLog", x.GetProgramLog);
        // without the driver library (a machine with no GPU) programs can still be compiled, not loaded
        if (drv)
            sym(drv, "cuModuleLoadData", x.ModuleLoadData), sym(drv, "cuModuleGetFunction", x.ModuleGetFunction),
                sym(drv, "cuLaunchKernelEx", x.LaunchKernelEx), sym(drv, "cuFuncSetAttribute", x.FuncSetAttribute),
                sym(drv, "cuOccupancyMaxActiveBlocksPerMultiprocessor", x.OccupancyMaxActiveBlocksPerMultiprocessor),
                sym(drv, "cuGetErrorString", x.GetErrorString), sym(drv, "cuOccupancyMaxActiveClusters", x.OccupancyMaxActiveClusters);
        x.ok = ok;
        return x;
    }();
    return a;
}

std::string program_struct(const JitProgram &p) {
    std::string s = "#include \"compiled_shells.cuh\"\nnamespace {\nstruct JP {\n    static constexpr const char *name = \"specialised\";\n";
    s += "    static constexpr int kind = " + std::to_string(p.kind) + ", flavour = " + std::to_string(p.flavour) + ", n_pro = " +
         std::to_string(p.n_pro) + ", n_ins = " + std::to_string(p.ins.size()) + ", n_slots = " + std::to_string(p.dtype.size()) + ";\n";
    s += "    static constexpr LtIns ins[" + std::to_string(p.ins.size()) + "] = {";
    for (size_t i = 0; i < p.ins.size(); ++i) s += (i ? ", {" : "{") + std::to_string(p.ins[i].op) + ", " + std::to_string(p.ins[i].imm) + "}";
    s += "};\n    static constexpr uint8_t dtype[" + std::to_string(p.dtype.size()) + "] = {";
    for (size_t i = 0; i < p.dtype.size(); ++i) s += (i ? ", " : "") + std::to_string(p.dtype[i]);
    s += "};\n    static constexpr uint8_t cls[" + std::to_string(p.cls.size()) + "] = {";
    for (size_t i = 0; i < p.cls.size(); ++i) s += (i ? ", " : "") + std::to_string(p.cls[i]);
    s += "};\n};\n}\n";
    return s;
}

// kernel instantiations one program needs: (name expression, slot in JitKernel::fn)
std::vector<std::pair<std::string, int>> variants_of(const JitProgram &p) {
    std::vector<std::pair<std::string, int>> v;
    if (p.kind == 0 && jit_reduced_slot(p) >= 0) v.push_back({"lt_c_ewred<JP>", 0});
    else if (p.kind == 0) v.push_back({"lt_c_ew<JP, 1>", 0});
    else if (p.kind == 2) v.push_back({std::string("lt_c_multi<JP, ") + (p.flavour == 2 ? "1" : "2") + ">", 0});
    else if (p.long_row) {
        v.push_back({"lt_c_longrow<JP, 256>", 0});
        v.push_back({"lt_c_longrow<JP, 512>", 1});
        if (p.cluster_u > 0) {
            v.push_back({"lt_c_rowc<JP, " + std::to_string(p.cluster_u) + ", false>", 2});
            if (jit_cluster_vector_bytes(p, 1) > 0) v.push_back({"lt_c_rowc<JP, " + std::to_string(p.cluster_u) + ", true>", 3});
        }
    } else {
        v.push_back({"lt_c_row<JP, " + std::to_string(p.row_u) + ">", 0});
    }
    return v;
}

// ---- optional on-disk cache of the machine code (environment variable LT_KERNEL_CACHE = a directory)
//
// A file per (program, library sources): "<hash>.ltk" = magic, the lowered kernel names, the machine code.  The
// hash covers the program's generated table entry and the text of the device headers, so a rebuilt library with
// changed shells never picks up stale code.  Files are written to a temporary name and renamed.

uint64_t fnv1a(const std::string &s, uint64_t h = 1469598103934665603ull) {
    for (unsigned char c : s) h = (h ^ c) * 1099511628211ull;
    return h;
}

std::string cache_path(const std::string &src, const JitProgram &p) {
    const char *dir = getenv("LT_KERNEL_CACHE");
    if (!dir || !*dir) return "";
    uint64_t h = fnv1a(src);
    for (const char *t : {kSrcVm, kSrcVmOps, kSrcPdl, kSrcShells}) h = fnv1a(t, h);
    h = fnv1a(std::string(p.long_row ? "L" : "R") + std::to_string(p.row_u) + "C" + std::to_string(p.cluster_u) + "/" + std::to_string(api().compiler_version), h);
    char name[64];
    snprintf(name, sizeof(name), "/%016llx.ltk", (unsigned long long)h);
    return std::string(dir) + name;
}

bool cache_read(const std::string &path, JitKernel &k) {
    FILE *f = fopen(path.c_str(), "rb");
    if (!f) return false;
    bool ok = false;
    uint32_t head[6] = {0, 0, 0, 0, 0, 0};  // magic, lengths of the four kernel names, length of the machine code
    if (fread(head, sizeof(head), 1, f) == 1 && head[0] == 0x4b544c33u && head[1] < 4096 && head[2] < 4096 && head[3] < 4096 &&
        head[4] < 4096 && head[5] > 0 && head[5] < (64u << 20)) {
        ok = true;
        for (int v = 0; v < 4 && ok; ++v) {
            k.entry[v].resize(head[1 + v]);
            ok = head[1 + v] == 0 || fread(&k.entry[v][0], head[1 + v], 1, f) == 1;
        }
        k.cubin.resize(head[5]);
        ok = ok && fread(k.cubin.data(), head[5], 1, f) == 1;
    }
    fclose(f);
    return ok;
}

void cache_write(const std::string &path, const JitKernel &k) {
    const std::string tmp = path + ".tmp" + std::to_string((unsigned long long)(uintptr_t)&k);
    FILE *f = fopen(tmp.c_str(), "wb");
    if (!f) return;
    const uint32_t head[6] = {0x4b544c33u, (uint32_t)k.entry[0].size(), (uint32_t)k.entry[1].size(), (uint32_t)k.entry[2].size(),
                              (uint32_t)k.entry[3].size(), (uint32_t)k.cubin.size()};
    bool ok = fwrite(head, sizeof(head), 1, f) == 1;
    for (int v = 0; v < 4 && ok; ++v) ok = k.entry[v].empty() || fwrite(k.entry[v].data(), k.entry[v].size(), 1, f) == 1;
    ok = ok && fwrite(k.cubin.data(), k.cubin.size(), 1, f) == 1;
    ok = fclose(f) == 0 && ok;
    if (ok) rename(tmp.c_str(), path.c_str());
    else remove(tmp.c_str());
}

void compile(JitKernel &k) {
    const Api &a = api();
    const std::string src = program_struct(k.program);
    const std::string cached = cache_path(src, k.program);
    if (!cached.empty() && cache_read(cached, k)) {
        k.log = "(machine code from " + cached + ")";
        k.state.store(1);
        return;
    }
    const char *names[] = {"vm.h", "vm_ops.cuh", "pdl.cuh", "compiled_shells.cuh"};
    const char *texts[] = {kSrcVm, kSrcVmOps, kSrcPdl, kSrcShells};
    nvrtcProgram prog = nullptr;
    if (a.CreateProgram(&prog, src.c_str(), "specialised.cu", 4, texts, names) != NVRTC_SUCCESS) {
        k.log = "nvrtcCreateProgram failed";
        k.state.store(-1);
        return;
    }
    const auto variants = variants_of(k.program);
    for (auto &v : variants) a.AddNameExpression(prog, v.first.c_str());
    // the log then carries the assembler's resource lines (registers, spills, shared memory) of every kernel
    const char *opts[] = {"--gpu-architecture=sm_100a", "-std=c++17", "-default-device", "-diag-suppress=177", "--ptxas-options=-v"};
    const nvrtcResult r = a.CompileProgram(prog, 5, opts);
    size_t n = 0;
    if (a.GetProgramLogSize(prog, &n) == NVRTC_SUCCESS && n > 1) {
        k.log.resize(n);
        a.GetProgramLog(prog, &k.log[0]);
    }
    bool ok = r == NVRTC_SUCCESS;
    if (ok) {
        for (auto &v : variants) {
            const char *low = nullptr;
            ok = ok && a.GetLoweredName(prog, v.first.c_str(), &low) == NVRTC_SUCCESS && low;
            if (ok) k.entry[v.second] = low;
        }
        ok = ok && a.GetCUBINSize(prog, &n) == NVRTC_SUCCESS && n > 0;
        if (ok) {
            k.cubin.resize(n);
            ok = a.GetCUBIN(prog, k.cubin.data()) == NVRTC_SUCCESS;
        }
    }
    a.DestroyProgram(&prog);
    if (getenv("LT_KERNEL_LOG")) fprintf(stderr, "[lazytensor] specialised %s (compiler %d):\n%s\n", variants.empty() ? "" : variants[0].first.c_str(), a.compiler_version, k.log.c_str());
    if (ok && !cached.empty()) cache_write(cached, k);
    k.state.store(ok ? 1 : -1);
}

// One worker thread for the whole process; jobs only produce machine code, so they outlive no context.
struct Worker {
    std::mutex m;
    std::condition_variable cv;
    std::deque<std::shared_ptr<JitKernel>> queue;
    std::map<std::string, std::shared_ptr<JitKernel>> cache;  // by program identity
    std::thread th;
    bool stop = false;
    ~Worker() {
        {
            std::lock_guard<std::mutex> g(m);
            stop = true;
            queue.clear();
        }
        cv.notify_all();
        if (th.joinable()) th.join();
    }
    void run() {
        for (;;) {
            std::shared_ptr<JitKernel> job;
            {
                std::unique_lock<std::mutex> g(m);
                cv.wait(g, [&] { return stop || !queue.empty(); });
                if (stop) return;
                job = queue.front();
                queue.pop_front();
            }
            compile(*job);
        }
    }
};

Worker &worker() {
    static Worker w;
    return w;
}

std::string identity(const JitProgram &p) {
    std::string s;
    s.push_back((char)p.kind);
    s.push_back((char)p.flavour);
    s.push_back((char)p.long_row);
    s.push_back((char)p.row_u);
    s.push_back((char)p.cluster_u);
    s.append((const char *)&p.n_pro, sizeof(p.n_pro));
    s.append((const char *)p.ins.data(), p.ins.size() * sizeof(LtIns));
    s.append((const char *)p.dtype.data(), p.dtype.size());
    s.append((const char *)p.cls.data(), p.cls.size());
    return s;
}

}  // namespace

bool jit_available() { return api().ok; }

std::shared_ptr<JitKernel> jit_request(const JitProgram &p, bool synchronous) {
    if (!api().ok) return nullptr;
    Worker &w = worker();
    std::shared_ptr<JitKernel> k;
    bool fresh = false;
    {
        std::lock_guard<std::mutex> g(w.m);
        auto it = w.cache.find(identity(p));
        if (it != w.cache.end()) k = it->second;
        else {
            k = std::make_shared<JitKernel>();
            k->program = p;
            w.cache[identity(p)] = k;
            fresh = true;
            if (!synchronous) {
                if (!w.th.joinable()) w.th = std::thread([&w] { w.run(); });
                w.queue.push_back(k);
            }
        }
    }
    if (fresh && synchronous) compile(*k);
    else if (fresh) w.cv.notify_one();
    else if (synchronous)
        while (k->state.load() == 0) std::this_thread::yield();  // someone else is compiling it: wait for them
    return k;
}

// ---- loading and launching (on the thread, and with the device, of the caller)

static const char *cu_text(CUresult r) {
    const char *s = nullptr;
    if (api().GetErrorString) api().GetErrorString(r, &s);
    return s ? s : "driver error";
}

bool jit_load(JitKernel &k, int device, std::string *err) {
    if (k.state.load() != 1) return false;
    std::lock_guard<std::mutex> g(k.load_lock);
    auto it = k.loaded.find(device);
    if (it != k.loaded.end()) return it->second.ok;
    JitKernel::Loaded L;
    const Api &a = api();
    if (!a.ModuleLoadData || !a.LaunchKernelEx) {
        if (err) *err = "the CUDA driver library is not available";
        k.loaded[device] = L;
        return false;
    }
    CUmodule mod = nullptr;
    CUresult r = a.ModuleLoadData(&mod, k.cubin.data());
    if (r == CUDA_SUCCESS) {
        L.ok = true;
        for (int v = 0; v < 4 && L.ok; ++v)
            if (!k.entry[v].empty()) {
                CUfunction f = nullptr;
                r = a.ModuleGetFunction(&f, mod, k.entry[v].c_str());
                L.ok = r == CUDA_SUCCESS;
                L.fn[v] = f;
            }
    }
    if (!L.ok && err) *err = std::string("loading a specialised kernel: ") + cu_text(r);
    k.loaded[device] = L;
    return L.ok;
}

static void *fn_of(JitKernel &k, int device, int variant) {
    std::lock_guard<std::mutex> g(k.load_lock);  // (contexts on other threads may be loading the same kernel on their device)
    auto it = k.loaded.find(device);
    return it == k.loaded.end() || !it->second.ok ? nullptr : it->second.fn[variant];
}

int jit_occupancy(JitKernel &k, int device, int variant, int threads, size_t dyn_smem) {
    CUfunction f = (CUfunction)fn_of(k, device, variant);
    if (!f) return 1;
    const Api &a = api();
    if (dyn_smem > 32u * 1024u) a.FuncSetAttribute(f, CU_FUNC_ATTRIBUTE_MAX_DYNAMIC_SHARED_SIZE_BYTES, (int)dyn_smem);
    int n = 0;
    if (a.OccupancyMaxActiveBlocksPerMultiprocessor(&n, f, threads, dyn_smem) != CUDA_SUCCESS || n < 1) n = 1;
    return n;
}

int jit_cluster_occupancy(JitKernel &k, int device, int variant, int threads, unsigned cluster, size_t dyn_smem) {
    CUfunction f = (CUfunction)fn_of(k, device, variant);
    const Api &a = api();
    if (!f || !a.OccupancyMaxActiveClusters) return 0;
    if (dyn_smem > 32u * 1024u) a.FuncSetAttribute(f, CU_FUNC_ATTRIBUTE_MAX_DYNAMIC_SHARED_SIZE_BYTES, (int)dyn_smem);
    CUlaunchConfig cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.sharedMemBytes = (unsigned)dyn_smem;
    cfg.gridDimX = cluster;
    cfg.gridDimY = cfg.gridDimZ = 1;
    cfg.blockDimX = (unsigned)threads;
    cfg.blockDimY = cfg.blockDimZ = 1;
    CUlaunchAttribute attr[1];
    memset(attr, 0, sizeof(attr));
    attr[0].id = CU_LAUNCH_ATTRIBUTE_CLUSTER_DIMENSION;
    attr[0].value.clusterDim.x = cluster;
    attr[0].value.clusterDim.y = attr[0].value.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (a.OccupancyMaxActiveClusters(&n, f, &cfg) != CUDA_SUCCESS) n = 0;
    return n;
}

bool jit_launch(JitKernel &k, int device, int variant, unsigned grid, unsigned threads, size_t dyn_smem, void *stream, void **args,
                std::string *err, unsigned cluster, unsigned grid_y) {
    CUfunction f = (CUfunction)fn_of(k, device, variant);
    if (!f) {
        if (err) *err = "specialised kernel not loaded";
        return false;
    }
    const Api &a = api();
    if (dyn_smem > 32u * 1024u) {
        const CUresult r = a.FuncSetAttribute(f, CU_FUNC_ATTRIBUTE_MAX_DYNAMIC_SHARED_SIZE_BYTES, (int)dyn_smem);
        if (r != CUDA_SUCCESS) {
            if (err) *err = std::string("cuFuncSetAttribute: ") + cu_text(r);
            return false;
        }
    }
    CUlaunchConfig cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDimX = grid;
    cfg.gridDimY = grid_y ? grid_y : 1;
    cfg.gridDimZ = 1;
    cfg.blockDimX = threads;
    cfg.blockDimY = cfg.blockDimZ = 1;
    cfg.sharedMemBytes = (unsigned)dyn_smem;
    cfg.hStream = (CUstream)stream;
    CUlaunchAttribute attr[2];
    memset(attr, 0, sizeof(attr));
    attr[0].id = CU_LAUNCH_ATTRIBUTE_PROGRAMMATIC_STREAM_SERIALIZATION;  // see pdl.cuh
    attr[0].value.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cluster) {
        attr[1].id = CU_LAUNCH_ATTRIBUTE_CLUSTER_DIMENSION;
        attr[1].value.clusterDim.x = cluster;
        attr[1].value.clusterDim.y = attr[1].value.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
    const CUresult r = a.LaunchKernelEx(&cfg, f, args, nullptr);
    if (r != CUDA_SUCCESS) {
        if (err) *err = std::string("cuLaunchKernelEx: ") + cu_text(r);
        return false;
    }
    return true;
}

// ---- what the executor needs to know about a program without instantiating anything (cf. Info<> in the shells)

static bool reads_slot(const LtIns &in) {
    return (in.op >= OP_LD && in.op < OP_LD + LT_VM_ND) || (in.op >= OP_F2M && in.op < OP_F2M + F2M_COUNT);
}

static size_t chunk_bytes(uint8_t dtype) { return dtype == LT_ST_BF16 ? 16 : dtype == LT_ST_U8 ? 8 : 32; }

size_t jit_row_stage_bytes(const JitProgram &p, int u, int threads) {
    size_t off = 0;
    for (size_t k = p.n_pro; k < p.ins.size(); ++k)
        if (reads_slot(p.ins[k]) && p.cls[p.ins[k].imm] == LT_CLS_FULL) off += chunk_bytes(p.dtype[p.ins[k].imm]) * (size_t)u * threads;
    return off;
}

bool jit_integer_heavy(const JitProgram &p) {
    for (const LtIns &in : p.ins)
        if (in.op == OP_PHILOX) return true;
    return false;
}

size_t jit_long_stage_bytes(const JitProgram &p, uint32_t cols) {
    size_t off = 0;
    for (size_t s = 0; s < p.dtype.size(); ++s) {
        if (p.cls[s] != LT_CLS_FULL) continue;
        bool in = false;
        for (size_t k = p.n_pro; k < p.ins.size() && !in; ++k) in = reads_slot(p.ins[k]) && p.ins[k].imm == s;
        if (!in) continue;
        const size_t es = p.dtype[s] == LT_ST_BF16 ? 2 : p.dtype[s] == LT_ST_U8 ? 1 : 4;
        if (((size_t)cols * es) % 16u) return 0;
        off += ((size_t)cols * es + 15u) & ~(size_t)15u;
    }
    return off;
}

int jit_reductions(const JitProgram &p) {
    int n = 0;
    for (size_t k = p.n_pro; k < p.ins.size(); ++k) n += p.ins[k].op >= OP_RED_SUM && p.ins[k].op <= OP_RED_MIN;
    return n;
}

int jit_reduced_slot(const JitProgram &p) {
    for (size_t s = 0; s < p.cls.size(); ++s)
        if (p.cls[s] >= LT_CLS_REDUCED) return (int)s;
    return -1;
}

size_t jit_cluster_vector_bytes(const JitProgram &p, int u) {
    bool reserved[LT_VM_NT] = {false};
    size_t n = 0;
    for (uint32_t k = 0; k < p.n_pro && k < p.ins.size(); ++k) {
        const int d = (int)p.ins[k].op - OP_LD;
        if (d >= 0 && d < LT_VM_NT && !reserved[d]) reserved[d] = true, ++n;
    }
    return n * (size_t)u * 128u * 32u;
}

// What the shells can express (cf. the checks of the table generator): broadcast operands loaded in the prologue into
// temporaries that nothing overwrites, results that are full-class or one value per row.
bool jit_supported(const JitProgram &p) {
    bool reserved[LT_VM_NT] = {false};
    for (uint32_t k = 0; k < p.n_pro; ++k) {
        const int d = (int)p.ins[k].op - OP_LD;
        if (d < 0 || d >= LT_VM_NT || p.cls[p.ins[k].imm] == LT_CLS_FULL) return false;
        reserved[d] = true;
    }
    for (size_t k = p.n_pro; k < p.ins.size(); ++k) {
        const uint32_t op = p.ins[k].op;
        if (op >= OP_MOV_T_ACC && op < OP_MOV_T_ACC + LT_VM_NT && reserved[op - OP_MOV_T_ACC]) return false;
        if (op >= OP_LD && op < OP_LD + LT_VM_NT && reserved[op - OP_LD]) return false;
        if (op == OP_ST && p.cls[p.ins[k].imm] != LT_CLS_FULL && p.cls[p.ins[k].imm] != LT_CLS_ROWVEC &&
            !(p.kind == 0 && p.cls[p.ins[k].imm] >= LT_CLS_REDUCED))
            return false;
    }
    return jit_reductions(p) <= 4;
}

}  // namespace lt
