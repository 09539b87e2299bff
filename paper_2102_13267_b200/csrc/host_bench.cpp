// Host-side cost of the path without Python: records, flushes and replays the graphs of three of the
// benchmark configurations through the C ABI on a record-and-plan-only context (no GPU needed: nothing is
// launched) and prints nanoseconds per barrier for each phase.
//
//   g++ -O2 -std=c++17 -I include paper_2102_13267_b200/csrc/host_bench.cpp \
//       -L paper_2102_13267_b200 -llazytensor -Wl,-rpath,$PWD/paper_2102_13267_b200 -o lt_host_bench && ./lt_host_bench
#include <chrono>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <initializer_list>
#include <vector>

#include "lazytensor.h"

namespace {

lt_ctx *ctx = nullptr;

void check(lt_status s, const char *what) {
    if (s != LT_OK) {
        fprintf(stderr, "%s: status %d: %s\n", what, (int)s, lt_last_error(ctx));
        exit(1);
    }
}

lt_tensor leaf(lt_dtype dt, std::vector<int64_t> shape) {
    static uintptr_t next = (uintptr_t)1 << 32;  // addresses that are never dereferenced
    next += (uintptr_t)1 << 28;
    lt_tensor t;
    check(lt_tensor_from_device(ctx, (void *)next, dt, (int)shape.size(), shape.data(), &t), "lt_tensor_from_device");
    return t;
}

lt_tensor scalar(double v) {
    lt_tensor t;
    check(lt_scalar(ctx, v, LT_F32, &t), "lt_scalar");
    return t;
}

// (initializer lists live on the stack: the harness itself allocates nothing per call)
lt_tensor op(int code, std::initializer_list<lt_tensor> in, std::initializer_list<int64_t> attrs = {}) {
    lt_tensor t;
    check(lt_op(ctx, code, in.begin(), (int)in.size(), attrs.size() ? attrs.begin() : nullptr, (int)attrs.size(), &t), "lt_op");
    return t;
}

// records the op, then releases the operands marked temporary (what a front end's reference counting does)
lt_tensor op_t(int code, std::initializer_list<lt_tensor> in, std::initializer_list<int> temp, std::initializer_list<int64_t> attrs = {}) {
    lt_tensor t = op(code, in, attrs);
    for (int i : temp) check(lt_release(ctx, in.begin()[i]), "lt_release");
    return t;
}

double now() { return std::chrono::duration<double>(std::chrono::steady_clock::now().time_since_epoch()).count(); }

void report(const char *name, int steps, double sec) {
    lt_stats st;
    lt_get_stats(ctx, &st);
    const double b = (double)(st.barriers ? st.barriers : 1);
    printf("%-28s %8.2f us/step | per barrier: record %7.0f ns, canonicalise %7.0f, hash+lookup %6.0f, plan %6.0f, bind+launch %6.0f, "
           "rebind %6.0f | nodes %llu, compiles %llu, hits %llu (%llu by matched trace, %llu traces diverged), replays %llu\n",
           name, 1e6 * sec / steps, st.ns_record / b, st.ns_canonicalise / b, st.ns_hash_lookup / b, st.ns_plan / b,
           st.ns_bind_launch / (b + (double)st.replays), st.ns_rebind / (b + (double)st.replays), (unsigned long long)st.nodes_recorded,
           (unsigned long long)st.compiles, (unsigned long long)st.cache_hits, (unsigned long long)st.traces_matched,
           (unsigned long long)st.traces_diverged, (unsigned long long)st.replays);
}

void elementwise_chain(int steps) {
    lt_tensor a = leaf(LT_F32, {1024, 1024}), b = leaf(LT_F32, {1024, 1024}), c = leaf(LT_F32, {1024, 1024}),
              d = leaf(LT_F32, {1024, 1024});
    lt_reset_stats(ctx);
    const double t0 = now();
    for (int i = 0; i < steps; ++i) {
        lt_tensor t = op(LT_OP_MUL, {a, b});
        t = op_t(LT_OP_ADD, {t, c}, {0});
        t = op_t(LT_OP_RELU, {t}, {0});
        t = op_t(LT_OP_MUL, {t, scalar(0.5)}, {0, 1});
        lt_tensor y = op_t(LT_OP_SUB, {t, d}, {0});
        check(lt_barrier(ctx, 0), "lt_barrier");
        check(lt_release(ctx, y), "lt_release");
    }
    report("C1 elementwise chain", steps, now() - t0);
}

void mlp_epilogue(int steps) {
    lt_tensor x = leaf(LT_BF16, {8192, 4096}), h = leaf(LT_BF16, {8192, 4096}), bias = leaf(LT_BF16, {4096});
    lt_reset_stats(ctx);
    const double t0 = now();
    for (int i = 0; i < steps; ++i) {
        lt_tensor xf = op(LT_OP_CONVERT, {x}, {LT_F32}), hf = op(LT_OP_CONVERT, {h}, {LT_F32}), bf = op(LT_OP_CONVERT, {bias}, {LT_F32});
        lt_tensor t = op_t(LT_OP_ADD, {hf, bf}, {0, 1});
        t = op_t(LT_OP_GELU_TANH, {t}, {0});
        t = op_t(LT_OP_ADD, {xf, t}, {0, 1});
        lt_tensor y = op_t(LT_OP_CONVERT, {t}, {0}, {LT_BF16});
        check(lt_barrier(ctx, 0), "lt_barrier");
        check(lt_release(ctx, y), "lt_release");
    }
    report("C2 MLP epilogue", steps, now() - t0);
}

struct Adam {
    std::vector<lt_tensor> p, g, m, v;
    lt_tensor beta1, omb1, beta2, omb2, sqrt_bc2, eps, step_size;
    void scalars(int step) {
        beta1 = scalar(0.9); omb1 = scalar(1.0 - 0.9); beta2 = scalar(0.999); omb2 = scalar(1.0 - 0.999);
        sqrt_bc2 = scalar(std::sqrt(1.0 - std::pow(0.999, step))); eps = scalar(1e-8);
        step_size = scalar(1e-3 / (1.0 - std::pow(0.9, step)));
    }
    void release_scalars() {
        for (lt_tensor s : {beta1, omb1, beta2, omb2, sqrt_bc2, eps, step_size}) check(lt_release(ctx, s), "lt_release");
    }
    void record() {
        for (size_t i = 0; i < p.size(); ++i) {
            lt_tensor m_new = op_t(LT_OP_ADD, {op(LT_OP_MUL, {m[i], beta1}), op(LT_OP_MUL, {g[i], omb1})}, {0, 1});
            lt_tensor gg = op(LT_OP_MUL, {g[i], g[i]});
            lt_tensor v_new = op_t(LT_OP_ADD, {op(LT_OP_MUL, {v[i], beta2}), op_t(LT_OP_MUL, {gg, omb2}, {0})}, {0, 1});
            lt_tensor den = op_t(LT_OP_ADD, {op_t(LT_OP_DIV, {op(LT_OP_SQRT, {v_new}), sqrt_bc2}, {0}), eps}, {0});
            lt_tensor upd = op_t(LT_OP_MUL, {op_t(LT_OP_DIV, {m_new, den}, {1}), step_size}, {0});
            lt_tensor p_new = op_t(LT_OP_SUB, {p[i], upd}, {1});
            check(lt_assign(ctx, m[i], m_new), "lt_assign");
            check(lt_assign(ctx, v[i], v_new), "lt_assign");
            check(lt_assign(ctx, p[i], p_new), "lt_assign");
            for (lt_tensor t : {m_new, v_new, p_new}) check(lt_release(ctx, t), "lt_release");
        }
    }
};

// the 161 parameter shapes of ResNet-50 (element counts only matter here)
std::vector<int64_t> resnet50_numels() {
    std::vector<int64_t> n;
    auto conv_bn = [&n](int64_t cout, int64_t cin, int64_t k) {
        n.push_back(cout * cin * k * k);
        n.push_back(cout);
        n.push_back(cout);
    };
    conv_bn(64, 3, 7);
    int64_t in = 64;
    const int blocks[4] = {3, 4, 6, 3}, widths[4] = {64, 128, 256, 512};
    for (int s = 0; s < 4; ++s)
        for (int b = 0; b < blocks[s]; ++b) {
            const int64_t w = widths[s];
            conv_bn(w, in, 1);
            conv_bn(w, w, 3);
            conv_bn(4 * w, w, 1);
            if (b == 0) conv_bn(4 * w, in, 1);
            in = 4 * w;
        }
    n.push_back(1000 * 2048);
    n.push_back(1000);
    return n;
}

// the same update as one lt_op_many call per parameter
void adam_batched(int steps) {
    Adam A;
    for (int64_t ne : resnet50_numels()) {
        A.p.push_back(leaf(LT_F32, {ne}));
        A.g.push_back(leaf(LT_F32, {ne}));
        A.m.push_back(leaf(LT_F32, {ne}));
        A.v.push_back(leaf(LT_F32, {ne}));
    }
    // inputs: 0 p, 1 g, 2 m, 3 v, 4 beta1, 5 1-beta1, 6 beta2, 7 1-beta2, 8 sqrt_bc2, 9 eps, 10 step_size; results by entry: -(k+1)
    const lt_batch_op ops[16] = {
        {LT_OP_MUL, 2, {2, 4, 0}, 0, 0, 0},   {LT_OP_MUL, 2, {1, 5, 0}, 0, 0, 0},   {LT_OP_ADD, 2, {-1, -2, 0}, 0, 0, 0},  // m_new = entry 2
        {LT_OP_MUL, 2, {1, 1, 0}, 0, 0, 0},   {LT_OP_MUL, 2, {3, 6, 0}, 0, 0, 0},   {LT_OP_MUL, 2, {-4, 7, 0}, 0, 0, 0},
        {LT_OP_ADD, 2, {-5, -6, 0}, 0, 0, 0},                                                                              // v_new = entry 6
        {LT_OP_SQRT, 1, {-7, 0, 0}, 0, 0, 0}, {LT_OP_DIV, 2, {-8, 8, 0}, 0, 0, 0},  {LT_OP_ADD, 2, {-9, 9, 0}, 0, 0, 0},   // den = entry 9
        {LT_OP_DIV, 2, {-3, -10, 0}, 0, 0, 0}, {LT_OP_MUL, 2, {-11, 10, 0}, 0, 0, 0}, {LT_OP_SUB, 2, {0, -12, 0}, 0, 0, 0}, // p_new = entry 12
        {LT_BATCH_ASSIGN, 2, {2, -3, 0}, 0, 0, 0}, {LT_BATCH_ASSIGN, 2, {3, -7, 0}, 0, 0, 0}, {LT_BATCH_ASSIGN, 2, {0, -13, 0}, 0, 0, 0}};
    lt_reset_stats(ctx);
    const double t0 = now();
    for (int step = 1; step <= steps; ++step) {
        A.scalars(step);
        for (size_t i = 0; i < A.p.size(); ++i) {
            const lt_tensor in[11] = {A.p[i], A.g[i], A.m[i], A.v[i], A.beta1, A.omb1, A.beta2, A.omb2, A.sqrt_bc2, A.eps, A.step_size};
            lt_tensor res[16];
            check(lt_op_many(ctx, ops, 16, in, 11, nullptr, res), "lt_op_many");
        }
        A.release_scalars();
        check(lt_barrier(ctx, 0), "lt_barrier");
    }
    char name[64];
    snprintf(name, sizeof(name), "C5 Adam, %zu tensors, batched", A.p.size());
    report(name, steps, now() - t0);
}

void adam(int steps, bool replay) {
    Adam A;
    for (int64_t ne : resnet50_numels()) {
        A.p.push_back(leaf(LT_F32, {ne}));
        A.g.push_back(leaf(LT_F32, {ne}));
        A.m.push_back(leaf(LT_F32, {ne}));
        A.v.push_back(leaf(LT_F32, {ne}));
    }
    lt_reset_stats(ctx);
    const double t0 = now();
    if (!replay) {
        for (int step = 1; step <= steps; ++step) {
            A.scalars(step);
            A.record();
            A.release_scalars();
            check(lt_barrier(ctx, 0), "lt_barrier");
        }
    } else {
        A.scalars(1);
        A.record();
        check(lt_barrier(ctx, 0), "lt_barrier");
        for (int step = 2; step <= steps; ++step) {
            check(lt_scalar_set(ctx, A.sqrt_bc2, std::sqrt(1.0 - std::pow(0.999, step))), "lt_scalar_set");
            check(lt_scalar_set(ctx, A.step_size, 1e-3 / (1.0 - std::pow(0.9, step))), "lt_scalar_set");
            check(lt_replay(ctx, 0), "lt_replay");
        }
    }
    char name[64];
    snprintf(name, sizeof(name), "C5 Adam, %zu tensors%s", A.p.size(), replay ? ", replayed" : "");
    report(name, steps, now() - t0);
}

}  // namespace

int main() {
    check(lt_ctx_create(LT_DEVICE_NONE, nullptr, nullptr, &ctx), "lt_ctx_create");
    elementwise_chain(20000);
    mlp_epilogue(20000);
    adam(1000, false);
    adam_batched(1000);
    adam(1000, true);
    lt_ctx_destroy(ctx);
    return 0;
}
