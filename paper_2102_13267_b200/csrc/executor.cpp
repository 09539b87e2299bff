// Executor: binds this trace's pointers and run-time scalars into a plan's parameter blocks
// and launches its kernels on the context's stream.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <memory>
#include <string>

#include "compiled.h"
#include "engine.h"
#include "launch.h"

namespace lt {

namespace {

uint32_t f32_bits(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    return u;
}

uint32_t encode_imm(const Imm &im, const std::vector<DynValue> &dyn) {
    if (im.enc == ENC_LO32 || im.enc == ENC_HI32) {
        uint64_t v = (uint64_t)dyn[im.dyn].i;
        return im.enc == ENC_LO32 ? (uint32_t)v : (uint32_t)(v >> 32);
    }
    const double v = im.dyn >= 0 ? dyn[im.dyn].d : im.sval;
    switch (im.enc) {
    case ENC_F32: return f32_bits((float)v);
    case ENC_BF16: {
        uint32_t u = f32_bits((float)v);
        if ((u & 0x7fffffffu) > 0x7f800000u) return u | 0x00400000u;
        u += 0x7fffu + ((u >> 16) & 1u);
        return u & 0xffff0000u;
    }
    case ENC_I32: return (uint32_t)(int32_t)(int64_t)v;
    case ENC_U8: return (uint32_t)(int64_t)v & 0xffu;
    default: return (uint32_t)(int64_t)v;
    }
}

cudaEvent_t take_event(lt_ctx *c) {
    if (!c->event_pool.empty()) {
        cudaEvent_t e = c->event_pool.back();
        c->event_pool.pop_back();
        return e;
    }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
}

bool aligned_for(uint64_t p, uint8_t dtype) { return (p & (dtype == LT_U8 ? 7u : 15u)) == 0; }

// The straight-line kernel of a launch comes from the build-time table (L.compiled) or from the run-time
// specialiser (L.jit, once its machine code is ready and loaded); the helpers below hide which.
bool specialised(const Launch &L) { return L.compiled < 0; }

// resident blocks per SM of a compiled kernel variant, asked once per plan launch
int compiled_blocks(lt_ctx *c, Launch &L, int u, int threads, size_t dyn = 0) {
    int lg = 0;
    while ((1 << lg) < u) ++lg;
    if (L.compiled_blocks[lg] == 0) {
        int b = 0;
        if (specialised(L)) b = jit_occupancy(*L.jit, c->device, 0, threads, dyn);
        else if (lt_compiled_occupancy(L.compiled, u, threads, dyn, &b) != cudaSuccess || b < 1) {
            cudaGetLastError();
            b = 1;
        }
        L.compiled_blocks[lg] = b;
    }
    return L.compiled_blocks[lg];
}

cudaError_t fast_launch(lt_ctx *c, Launch &L, const void *params, int u, unsigned grid, unsigned threads, unsigned group, unsigned group_log2,
                        unsigned depth, size_t dyn) {
    if (!specialised(L)) return lt_compiled_launch(L.compiled, params, u, grid, threads, group, group_log2, depth, c->stream);
    uint32_t a1 = group, a2 = group_log2, a3 = depth;
    void *args[4] = {const_cast<void *>(params), &a1, &a2, &a3};
    std::string err;
    if (!jit_launch(*L.jit, c->device, 0, grid, threads, dyn, (void *)c->stream, args, &err)) {
        c->error = err;
        return cudaErrorLaunchFailure;
    }
    c->stats.launches_specialised++;
    return cudaSuccess;
}

// Is there a straight-line kernel for this launch right now?  Requests the specialisation when the plan has run
// often enough, and loads its machine code when it has arrived.
bool fast_kernel_ready(lt_ctx *c, Launch &L) {
    if (!c->opt.compiled) return false;
    if (L.compiled >= 0) return true;
    if (!L.jit_program || L.jit_failed || !c->opt.specialise) return false;
    ++L.runs;
    if (!L.jit) {
        const bool now = c->opt.specialise == 1;
        if (!now && (int64_t)L.runs < c->opt.specialise_after) return false;
        L.jit = jit_request(*L.jit_program, now);
        if (!L.jit) {
            L.jit_failed = true;
            return false;
        }
        c->stats.programs_specialised++;
    }
    const int st = L.jit->state.load();
    if (st == 0) return false;  // still being compiled: the interpreter serves this flush
    std::string err;
    if (st < 0 || !jit_load(*L.jit, c->device, &err)) {
        L.jit_failed = true;
        if (c->opt.log >= 1) fprintf(stderr, "[lazytensor] run-time specialisation failed: %s\n%s\n", err.c_str(), L.jit->log.c_str());
        return false;
    }
    return true;
}

}  // namespace

// Runs `plan`, or -- when one of its fused long-row launches cannot run on the pointers of this flush -- the
// same graph planned with every long row reduction as a kernel of its own.  *ran is the plan that was executed
// (its outputs' placement is what the caller binds).
lt_status run_plan(lt_ctx *c, Plan *plan, const Canonical &cg, Plan **ran) {
    bool needs_split = false;
    *ran = plan;
    lt_status s = execute_plan(c, *plan, cg, &needs_split);
    if (!needs_split) return s;
    if (!plan->split) {
        std::unique_ptr<Plan> sp(new Plan());
        s = build_plan(c, cg, *sp, true);
        if (s) return s;
        plan->split = std::move(sp);
    }
    *ran = plan->split.get();
    return execute_plan(c, *plan->split, cg, nullptr);
}

// A fused long-row launch, and an elementwise launch that reduces its result, run only on their compiled kernels,
// which need 128-bit accesses: whole chunks per row and 16-byte aligned inputs (results and temporaries come from
// the allocator, aligned).  Fills c->param_ptr.
bool long_rows_runnable(lt_ctx *c, Plan &plan, const Canonical &cg) {
    c->param_ptr.resize(plan.n_params);
    for (uint32_t i = 0; i < plan.n_params; ++i)
        c->param_ptr[i] = c->buffers[c->nodes[cg.param_node[i]].buffer].ptr;
    if (c->device == LT_DEVICE_NONE) return true;
    for (Launch &L : plan.launches) {
        const Group &g = plan.groups[L.groups[0]];
        if (!(L.kind == K_ROW && g.long_row) && !(L.kind == K_EW && g.fused_red)) continue;
        if (L.compiled < 0 && L.jit_program && !L.jit_failed && c->opt.compiled && c->opt.specialise == 2) {
            // no kernel in the table: ask the specialiser once the plan keeps coming back, and use the kernel when it is there
            if (!L.jit && (int64_t)++L.runs >= c->opt.specialise_after) {
                L.jit = jit_request(*L.jit_program, false);
                if (L.jit) c->stats.programs_specialised++;
                else L.jit_failed = true;
            }
            if (L.jit && L.jit->state.load() < 0) L.jit_failed = true;
        }
        const bool have_kernel = L.compiled >= 0 || (L.jit && !L.jit_failed && L.jit->state.load() == 1);
        bool ok = c->opt.compiled && have_kernel && (g.cols % LT_VM_V) == 0;
        for (size_t q = 0; q < g.io.size() && ok; ++q)
            if (g.io[q].kind == IO_PARAM && (g.io[q].cls <= LT_CLS_COLVEC || g.io[q].cls == LT_CLS_PITCHED))
                ok = aligned_for((uint64_t)(uintptr_t)c->param_ptr[g.io[q].index] + g.io[q].offset * dtype_size(g.io[q].dtype), g.io[q].dtype) &&
                     aligned_for((uint64_t)g.io[q].pitch * dtype_size(g.io[q].dtype), g.io[q].dtype);
        if (!ok) return false;
    }
    return true;
}

lt_status execute_plan(lt_ctx *c, Plan &plan, const Canonical &cg, bool *needs_split) {
    const bool dry = c->device == LT_DEVICE_NONE;
    const size_t n_out = plan.outputs.size();
    // Checked before anything is obtained or enqueued, so that the caller can fall back to the split plan.
    if (!long_rows_runnable(c, plan, cg)) {
        if (needs_split) {
            *needs_split = true;
            return LT_OK;
        }
        return fail(c, LT_ERR_UNSUPPORTED, "a fused reduction over rows of more than 8192 elements needs 16-byte aligned inputs and rows that are a multiple of 8 elements");
    }
    c->out_ptr.assign(n_out, nullptr);
    c->temp_ptr.assign(plan.temp_bytes.size(), nullptr);

    auto release_all = [&](bool outputs_too) {
        for (void *&p : c->temp_ptr) {
            if (p && !c->static_mode) ctx_free(c, p);
            p = nullptr;
        }
        if (outputs_too)
            for (size_t k = 0; k < n_out; ++k)
                if (c->out_ptr[k] && plan.outputs[k].donated_param < 0) {
                    ctx_free(c, c->out_ptr[k]);
                    c->out_ptr[k] = nullptr;
                }
    };

    if (c->static_mode) {
        // Allocation-free flush: every result must land in a buffer the caller handed in, every
        // parameter must be caller memory (so that nothing is returned to the allocator when the
        // graph is dropped), and the temporaries must fit the fixed scratch range.
        for (size_t k = 0; k < n_out; ++k)
            if (plan.outputs[k].donated_param < 0)
                return fail(c, LT_ERR_UNSUPPORTED,
                            "lt_barrier_static_scratch: a result has no caller buffer to go to (lt_assign it to an "
                            "input of the graph made by lt_tensor_from_device that no other tensor names)");
        for (uint32_t i = 0; i < plan.n_params; ++i)
            if (c->buffers[c->nodes[cg.param_node[i]].buffer].owned)
                return fail(c, LT_ERR_UNSUPPORTED, "lt_barrier_static_scratch: an input lives in library-owned memory");
        size_t need = 0;
        for (size_t t = 0; t < plan.temp_bytes.size(); ++t) need += (plan.temp_bytes[t] + 255u) & ~(size_t)255u;
        if (need > c->static_cap)
            return fail(c, LT_ERR_UNSUPPORTED, "lt_barrier_static_scratch: the graph needs " + std::to_string(need) +
                                                   " bytes of temporaries, the static scratch array holds " +
                                                   std::to_string(c->static_cap));
        if (c->static_clear && !dry) {
            cudaError_t ce = lt_static_scratch_clear_enqueue(c->static_base, c->static_cap, c->sm_count, c->stream);
            if (ce != cudaSuccess) return fail(c, LT_ERR_CUDA, std::string("clearing the static scratch: ") + cudaGetErrorString(ce));
        }
    }
    uint64_t donated = 0, allocated = 0;
    for (size_t k = 0; k < n_out; ++k) {
        const OutputPlan &o = plan.outputs[k];
        if (o.donated_param >= 0) {
            c->out_ptr[k] = c->param_ptr[o.donated_param];
            ++donated;
        } else {
            c->out_ptr[k] = ctx_alloc(c, o.bytes);
            if (!c->out_ptr[k]) {
                release_all(true);
                return fail(c, LT_ERR_OOM, "allocator returned null for an output");
            }
            ++allocated;
        }
    }
    size_t static_used = 0;
    for (size_t t = 0; t < plan.temp_bytes.size(); ++t) {
        if (c->static_mode) {
            c->temp_ptr[t] = (char *)c->static_base + static_used;
            static_used += (plan.temp_bytes[t] + 255u) & ~(size_t)255u;
            continue;
        }
        c->temp_ptr[t] = ctx_alloc(c, plan.temp_bytes[t]);
        if (!c->temp_ptr[t]) {
            release_all(true);
            return fail(c, LT_ERR_OOM, "allocator returned null for a temporary");
        }
    }

    auto resolve = [&](const IoRef &io) -> uint64_t {
        void *p = io.kind == IO_PARAM ? c->param_ptr[io.index] : io.kind == IO_OUTPUT ? c->out_ptr[io.index] : c->temp_ptr[io.index];
        return (uint64_t)(uintptr_t)p + io.offset * dtype_size(io.dtype);  // (offset: a slice read in place)
    };

    const unsigned waves = (unsigned)std::max<int64_t>(1, c->opt.waves);
    for (Launch &L : plan.launches) {
        cudaError_t e = cudaSuccess;
        cudaEvent_t ev0 = nullptr, ev1 = nullptr;
        if (c->timing && !dry) {
            ev0 = take_event(c);
            ev1 = take_event(c);
        }
        if (L.kind == K_VIEW) {
            const Group &g = plan.groups[L.groups[0]];
            unsigned launched = 1;
            if (!dry) {
                const IoRef &res = g.io.back();
                const bool upd = g.view_op == LT_OP_UPDATE_SLICE;
                const bool in_place = upd && res.kind == IO_OUTPUT && plan.outputs[res.index].donated_param >= 0 &&
                                      resolve(res) == resolve(g.io[0]);
                if (ev0) cudaEventRecord(ev0, c->stream);
                e = lt_launch_view(g.view_op, (int)dtype_size(res.dtype), g.view_rank, g.view_in_dims, g.view_out_dims, g.view_a0, g.view_a1,
                                   (const void *)(uintptr_t)resolve(g.io[0]), upd ? (const void *)(uintptr_t)resolve(g.io[1]) : nullptr,
                                   (void *)(uintptr_t)resolve(res), in_place ? 1 : 0, c->sm_count, c->stream, &launched);
                if (ev1) cudaEventRecord(ev1, c->stream);
            }
            c->stats.launches_view += 1;
            if (launched > 1) c->stats.kernels_launched += launched - 1;
        } else if (L.kind == K_RED) {
            const Group &g = plan.groups[L.groups[0]];
            unsigned launched = 1;
            if (!dry) {
                void *scratch = g.scratch_temp >= 0 ? c->temp_ptr[g.scratch_temp] : nullptr;
                if (ev0) cudaEventRecord(ev0, c->stream);
                if (g.from_partials)  // the kernel that computed the input left the first stage's partial results in scratch
                    e = lt_launch_reduce_final(g.red_axis, g.red_kind, g.io[1].dtype, scratch, (void *)(uintptr_t)resolve(g.io[1]),
                                               lt_reduce_parts(g.red_axis, g.rows, g.cols, c->sm_count), g.cols, c->stream);
                else
                    e = lt_launch_reduce(g.red_axis, g.red_kind, g.io[0].dtype, (const void *)(uintptr_t)resolve(g.io[0]),
                                         (void *)(uintptr_t)resolve(g.io[1]), scratch, g.rows, g.cols, c->sm_count, c->stream, &launched);
                if (ev1) cudaEventRecord(ev1, c->stream);
            }
            c->stats.launches_reduce += 1;
            if (launched > 1) c->stats.kernels_launched += launched - 1;
        } else if (L.kind == K_MULTI) {
            LtMultiParams &P = *L.mp;
            const Group &g0 = plan.groups[L.groups[0]];
            for (size_t q = 0; q < g0.imms.size(); ++q) P.scal[q] = encode_imm(g0.imms[q], cg.dyn);
            const size_t slots = g0.io.size();
            for (size_t k = 0; k < L.groups.size(); ++k) {
                const Group &g = plan.groups[L.groups[k]];
                for (size_t s = 0; s < slots; ++s) P.ptr[k * slots + s] = resolve(g.io[s]);
            }
            // staging plan: a slot is staged when its pointer is aligned in every instance
            {
                uint32_t pieces = 0;
                for (size_t s = 0; s < LT_VM_MAX_PTR; ++s) P.io_stage[s] = 0xff;
                if (c->opt.stage) {
                    for (size_t s = 0; s < slots; ++s) {
                        if (g0.io[s].is_store) continue;
                        const uint64_t need = g0.io[s].dtype == LT_U8 ? 7u : 15u;
                        bool ok = true;
                        for (size_t k = 0; k < L.groups.size() && ok; ++k) ok = (P.ptr[k * slots + s] & need) == 0;
                        if (!ok) continue;
                        P.io_stage[s] = (uint8_t)pieces;
                        pieces += (g0.io[s].dtype == LT_BF16 || g0.io[s].dtype == LT_U8) ? 1u : 2u;
                    }
                }
                P.stage_pieces = pieces;
                P.stage_depth = 0;
                if (pieces) {
                    const uint32_t buf = pieces * LT_VM_STAGE_PIECE;
                    uint32_t depth = (96u * 1024u + (uint32_t)c->occ_multi * buf - 1) / ((uint32_t)c->occ_multi * buf);
                    depth = std::min(4u, std::max(2u, depth));
                    while (depth >= 1 && depth * buf > LT_MAX_STAGE_BYTES) --depth;
                    // with fewer than three buffers the kernel also prefetches one chunk further into L2
                    if (depth >= (uint32_t)std::max<int64_t>(1, c->opt.stage)) P.stage_depth = depth;
                    else {
                        P.stage_pieces = 0;
                        for (size_t s = 0; s < LT_VM_MAX_PTR; ++s) P.io_stage[s] = 0xff;
                    }
                }
            }
            bool done = false;
            if (!dry && fast_kernel_ready(c, L)) {
                // compiled kernel: needs 128-bit accesses everywhere (aligned pointers, whole chunks)
                bool ok = true;
                for (size_t k = 0; k < L.groups.size() && ok; ++k) {
                    ok = (P.numel[k] % LT_VM_V) == 0;
                    for (size_t s = 0; s < slots && ok; ++s) ok = aligned_for(P.ptr[k * slots + s], g0.io[s].dtype);
                }
                if (ok) {
                    // two chunks in flight per thread and eight waves of blocks measured best for wide programs
                    // (four input streams) over many tensors of uneven size
                    // (one chunk with correctly rounded division and square root: their slow paths cost registers)
                    const int u = (c->opt.compiled_u > 0 && !specialised(L)) ? (int)c->opt.compiled_u : (L.flavour == 2 ? 1 : 2);
                    const int occ = compiled_blocks(c, L, u, LT_EW_THREADS);
                    const unsigned mwaves = c->opt.waves > 0 ? waves : 8u;  // (eight waves measured a few per cent faster than two on 161 tensors of uneven size)
                    unsigned grid = (unsigned)std::min<uint64_t>(P.total_super, (uint64_t)c->sm_count * occ * mwaves);
                    if (grid < 1) grid = 1;
                    if (ev0) cudaEventRecord(ev0, c->stream);
                    e = fast_launch(c, L, &P, u, grid, LT_EW_THREADS, 0, 0, 0, 0);
                    if (ev1) cudaEventRecord(ev1, c->stream);
                    c->stats.launches_compiled++;
                    done = true;
                }
            }
            if (!dry && !done) {
                unsigned grid = (unsigned)std::min<uint64_t>(P.total_super, (uint64_t)c->sm_count * c->occ_multi * waves);
                if (grid < 1) grid = 1;
                if (ev0) cudaEventRecord(ev0, c->stream);
                e = lt_launch_multi(P, L.flavour, grid, c->stream);
                if (ev1) cudaEventRecord(ev1, c->stream);
            }
            c->stats.launches_multi++;
        } else {
            LtKParams &P = *L.kp;
            const Group &g = plan.groups[L.groups[0]];
            for (size_t q = 0; q < g.imms.size(); ++q) P.scal[q] = encode_imm(g.imms[q], cg.dyn);
            for (size_t s = 0; s < g.io.size(); ++s) P.ptr[s] = resolve(g.io[s]);
            if (!g.long_row) {
                // Staging plan: aligned full-class inputs are copied asynchronously into per-thread
                // shared-memory buffers a few chunks ahead.  Needs rows that are a multiple of the chunk
                // (chunk c starts at element 8c) and 256-thread blocks (the buffer layout).
                const bool linear = L.kind == K_EW ? (!P.rowcol || (P.cols % LT_VM_V) == 0)
                                                   : ((P.cols % LT_VM_V) == 0 && L.threads == LT_EW_THREADS);
                const uint32_t occ = (uint32_t)(L.kind == K_EW ? c->occ_ew : c->occ_row);
                uint32_t pieces = 0;
                for (size_t s = 0; s < LT_VM_MAX_PTR; ++s) P.io_stage[s] = 0xff;
                if (c->opt.stage && linear) {
                    for (size_t s = 0; s < g.io.size(); ++s) {
                        const IoRef &io = g.io[s];
                        if (io.is_store || io.cls != LT_CLS_FULL) continue;
                        const uint64_t need = io.dtype == LT_U8 ? 7u : 15u;
                        if (P.ptr[s] & need) continue;
                        P.io_stage[s] = (uint8_t)pieces;
                        pieces += (io.dtype == LT_BF16 || io.dtype == LT_U8) ? 1u : 2u;
                    }
                }
                P.stage_pieces = pieces;
                P.stage_depth = 0;
                if (pieces) {
                    const uint32_t buf = pieces * LT_VM_STAGE_PIECE;
                    uint32_t depth = (96u * 1024u + occ * buf - 1) / (occ * buf);
                    depth = std::min(4u, std::max(2u, depth));
                    while (depth >= 1 && depth * buf > LT_MAX_STAGE_BYTES) --depth;
                    // iterations each thread runs: a launch that gives a thread one or two chunks gains nothing
                    // from look-ahead, but staging still fetches all its inputs in parallel
                    const uint64_t units = L.kind == K_EW ? (P.n_chunks + LT_EW_THREADS - 1) / LT_EW_THREADS
                                                          : ((uint64_t)P.rows + P.rows_per_cta - 1) / P.rows_per_cta;
                    const uint64_t resident = (uint64_t)c->sm_count * occ * waves;
                    const uint64_t iters = (units + resident - 1) / resident;
                    if (iters <= 2 && depth >= 1) depth = (uint32_t)std::min<uint64_t>(depth, iters);
                    // with fewer than three buffers the kernel also prefetches one chunk further into L2
                    if (depth >= (uint32_t)std::max<int64_t>(1, c->opt.stage) || (depth >= 1 && iters <= 2)) P.stage_depth = depth;
                    else {
                        P.stage_pieces = 0;
                        for (size_t s = 0; s < LT_VM_MAX_PTR; ++s) P.io_stage[s] = 0xff;
                    }
                }
            }
            bool done = false;
            if (g.fused_red) {
                // the group's kernel reduces one of its results: first stage here, second in the reduction group that follows
                if (!dry) {
                    if (specialised(L)) {
                        std::string err;
                        if (!jit_load(*L.jit, c->device, &err)) {
                            release_all(true);
                            return fail(c, LT_ERR_CUDA, err);
                        }
                    }
                    const unsigned parts = lt_reduce_parts(g.red_axis, g.rows, g.cols, c->sm_count);
                    const unsigned gx = g.red_axis == 1 ? (P.cpr + 31u) / 32u : parts, gy = g.red_axis == 1 ? parts : 1u;
                    uint32_t rows_per = (uint32_t)((g.rows + parts - 1) / parts);
                    if (ev0) cudaEventRecord(ev0, c->stream);
                    if (specialised(L)) {
                        void *args[2] = {&P, &rows_per};
                        std::string err;
                        if (!jit_launch(*L.jit, c->device, 0, gx, 256, 0, (void *)c->stream, args, &err, 0, gy)) {
                            c->error = err;
                            e = cudaErrorLaunchFailure;
                        } else {
                            c->stats.launches_specialised++;
                        }
                    } else {
                        e = lt_compiled_launch_reduced(L.compiled, &P, gx, gy, rows_per, c->stream);
                    }
                    if (ev1) cudaEventRecord(ev1, c->stream);
                }
                c->stats.launches_compiled++;
                done = true;
            } else if (g.long_row) {
                // a CTA per row, walking it in slices; rows staged in shared memory `depth` ahead when they fit
                // (feasibility was checked on entry)
                if (!dry && specialised(L)) {
                    std::string err;
                    if (!jit_load(*L.jit, c->device, &err)) {
                        release_all(true);
                        return fail(c, LT_ERR_CUDA, err);
                    }
                }
                // Up to 65536 columns: a thread-block cluster is the row's thread group and the row stays in registers
                // across the reductions (one pass over the data, column vectors loaded once per thread).
                unsigned cl_size = 0;
                int cl_u = 0;
                bool clustered = !dry && cluster_shape(P.cpr, g.n_pro > 0, c->opt.cluster, c->opt.compiled_row_u, &cl_size, &cl_u) &&
                                 (!specialised(L) || L.jit_program->cluster_u == cl_u);
                size_t cl_dyn = 0;
                unsigned cl_depth = 0;
                bool cl_shared = false;
                if (clustered) {
                    // column vectors that do not fit 64 registers per thread are kept in shared memory rather than re-read for every row
                    const size_t vec = specialised(L) ? jit_cluster_vector_bytes(*L.jit_program, cl_u) : lt_compiled_cluster_vector_bytes(L.compiled, cl_u);
                    cl_shared = vec > 0 && vec <= 160u * 1024u && (c->opt.cluster_vectors >= 0 ? c->opt.cluster_vectors != 0 : vec > 128u * 64u * 4u);
                    // the next rows' inputs travel through a ring of shared-memory stages: not for programs bound by integer
                    // issue, nor for 4-byte inputs, which measured faster loaded directly (softmax f32 at 65536 columns: 247 us
                    // against 333 with the ring; the requests of eight chunks per thread are in flight either way)
                    const size_t stage = specialised(L) ? jit_row_stage_bytes(*L.jit_program, cl_u, 128) : lt_compiled_row_stage_bytes(L.compiled, cl_u);
                    bool wants_ring = specialised(L) ? !jit_integer_heavy(*L.jit_program) : lt_compiled_prefers_staging(L.compiled) != 0;
                    for (size_t q = 0; q < g.io.size(); ++q)
                        if (!g.io[q].is_store && g.io[q].cls == LT_CLS_FULL && dtype_size(g.io[q].dtype) == 4) wants_ring = false;
                    cl_depth = c->opt.compiled_depth >= 0 ? (unsigned)c->opt.compiled_depth : (wants_ring ? 2u : 0u);
                    while (cl_depth > 0 && cl_depth * stage > 72u * 1024u) --cl_depth;
                    if (stage == 0) cl_depth = 0;
                    cl_dyn = cl_depth * stage + (cl_shared ? vec : 0);
                    if (L.cluster_max < 0) {
                        int n = 0;
                        if (specialised(L)) n = jit_cluster_occupancy(*L.jit, c->device, cl_shared ? 3 : 2, 128, cl_size, cl_dyn);
                        else if (lt_compiled_cluster_occupancy(L.compiled, cl_u, cl_shared ? 1 : 0, cl_size, cl_depth, &n) != cudaSuccess) {
                            cudaGetLastError();
                            n = 0;
                        }
                        L.cluster_max = n;
                    }
                    clustered = L.cluster_max >= 1;
                }
                if (clustered) {
                    const unsigned clusters = (unsigned)std::min<uint64_t>(P.rows, (uint64_t)L.cluster_max);
                    if (ev0) cudaEventRecord(ev0, c->stream);
                    if (specialised(L)) {
                        uint32_t a1 = cl_depth;
                        uint64_t a2 = (uint64_t)c->wait_limit_ns;
                        void *args[3] = {&P, &a1, &a2};
                        std::string err;
                        if (!jit_launch(*L.jit, c->device, cl_shared ? 3 : 2, clusters * cl_size, 128, cl_dyn, (void *)c->stream, args, &err, cl_size)) {
                            c->error = err;
                            e = cudaErrorLaunchFailure;
                        } else {
                            c->stats.launches_specialised++;
                        }
                    } else {
                        e = lt_compiled_launch_cluster(L.compiled, &P, cl_u, cl_shared ? 1 : 0, clusters, cl_size, cl_depth, (uint64_t)c->wait_limit_ns, c->stream);
                    }
                    if (ev1) cudaEventRecord(ev1, c->stream);
                    c->status_pending = true;
                }
                if (!dry && !clustered) {
                    // Staging and CTA size: the row a CTA works on is staged when it fits; several CTAs per SM overlap one
                    // another's passes; when a staged row leaves room for one CTA only, that CTA has 512 threads.
                    const size_t cap = 200u * 1024u;
                    const size_t stage = specialised(L) ? jit_long_stage_bytes(*L.jit_program, P.cols) : lt_compiled_long_stage_bytes(L.compiled, P.cols);
                    const unsigned deepest = stage == 0 ? 0u : (unsigned)std::min<size_t>(2, cap / stage);
                    auto blocks_at = [&](unsigned threads, unsigned d) {
                        int b = 0;
                        if (specialised(L)) b = jit_occupancy(*L.jit, c->device, threads >= 512 ? 1 : 0, (int)threads, d * stage);
                        else if (lt_compiled_long_occupancy(L.compiled, threads, d * stage, &b) != cudaSuccess || b < 1) {
                            cudaGetLastError();
                            b = 1;
                        }
                        return b;
                    };
                    // (one row ahead: two measured no faster, and the shared memory it takes is L1 the column vectors miss)
                    unsigned depth = std::min(deepest, 1u), threads = 256;
                    int occ = blocks_at(256, depth);
                    if (occ < 2 && depth >= 1) {
                        threads = 512;
                        occ = blocks_at(512, depth);
                    }
                    if (c->opt.compiled_depth >= 0 && (unsigned)c->opt.compiled_depth <= deepest) {
                        depth = (unsigned)c->opt.compiled_depth;
                        threads = c->opt.compiled_row_u == 512 ? 512 : 256;
                        occ = blocks_at(threads, depth);
                    }
                    unsigned grid = (unsigned)std::min<uint64_t>(P.rows, (uint64_t)c->sm_count * occ);
                    if (grid < 1) grid = 1;
                    // rows are multiples of 16 bytes when they can be staged; the request pays off when one CTA per SM
                    // leaves HBM idle during the passes that read shared memory only
                    bool l2_ahead = stage != 0 && occ < 2 && depth >= 1;
                    if (c->opt.long_l2_ahead >= 0) l2_ahead = stage != 0 && c->opt.long_l2_ahead != 0;
                    if (ev0) cudaEventRecord(ev0, c->stream);
                    if (specialised(L)) {
                        uint32_t a1 = depth, a2 = (uint32_t)stage, a4 = l2_ahead ? 1u : 0u;
                        uint64_t a3 = (uint64_t)c->wait_limit_ns;
                        void *args[5] = {&P, &a1, &a2, &a3, &a4};
                        std::string err;
                        if (!jit_launch(*L.jit, c->device, threads >= 512 ? 1 : 0, grid, threads, depth * stage, (void *)c->stream, args, &err)) {
                            c->error = err;
                            e = cudaErrorLaunchFailure;
                        } else {
                            c->stats.launches_specialised++;
                        }
                    } else {
                        e = lt_compiled_launch_long(L.compiled, &P, grid, threads, depth, stage, (uint64_t)c->wait_limit_ns, l2_ahead ? 1 : 0, c->stream);
                    }
                    if (ev1) cudaEventRecord(ev1, c->stream);
                    if (depth) c->status_pending = true;
                }
                c->stats.launches_compiled++;
                done = true;
            }
            if (!done && !dry && fast_kernel_ready(c, L)) {
                // compiled kernel: needs 128-bit accesses everywhere (aligned pointers, whole chunks)
                bool ok = (L.kind == K_EW && !P.rowcol) ? (P.n % LT_VM_V) == 0 : (P.cols % LT_VM_V) == 0;
                ok = ok && P.n_chunks < (1ull << 31);
                for (size_t s = 0; s < g.io.size() && ok; ++s) {
                    if (g.io[s].cls <= LT_CLS_COLVEC || g.io[s].cls == LT_CLS_PITCHED) ok = aligned_for(P.ptr[s], g.io[s].dtype);
                    if (ok && g.io[s].cls == LT_CLS_PITCHED) ok = aligned_for((uint64_t)g.io[s].pitch * dtype_size(g.io[s].dtype), g.io[s].dtype);
                }
                if (ok && L.kind == K_EW) {
                    // a tensor small enough for one wave of one-chunk CTAs runs on half as many CTAs with two chunks in flight
                    // per thread (measured on C1: 5.0 against 5.4 us); larger ones gain nothing from it
                    const uint64_t one_wave = (uint64_t)c->sm_count * (uint64_t)compiled_blocks(c, L, 1, LT_EW_THREADS);
                    const bool small = !specialised(L) && (P.n_chunks + LT_EW_THREADS - 1) / LT_EW_THREADS <= one_wave;
                    const int u = (c->opt.compiled_u > 0 && !specialised(L)) ? (int)c->opt.compiled_u : (small ? 2 : 1);
                    const int occ = compiled_blocks(c, L, u, LT_EW_THREADS);
                    const uint64_t need = (P.n_chunks + (uint64_t)LT_EW_THREADS * u - 1) / ((uint64_t)LT_EW_THREADS * u);
                    // a compiled CTA has no set-up to amortise: many short CTAs, scheduled by the hardware as others
                    // retire, beat one wave of persistent ones (measured; no change beyond 8 waves)
                    const unsigned ewaves = c->opt.waves > 0 ? waves : 16u;
                    unsigned grid = (unsigned)std::min<uint64_t>(need, (uint64_t)c->sm_count * occ * ewaves);
                    if (grid < 1) grid = 1;
                    if (ev0) cudaEventRecord(ev0, c->stream);
                    e = fast_launch(c, L, &P, u, grid, LT_EW_THREADS, 0, 0, 0, 0);
                    if (ev1) cudaEventRecord(ev1, c->stream);
                    done = true;
                } else if (ok && P.cpr <= 8u * 128u) {  // a row's group of threads is at most one CTA of 128
                    // a row lives in the registers of its thread group: up to 8 chunks per thread, one warp per row if it fits
                    bool four_byte = false;
                    for (size_t q = 0; q < g.io.size(); ++q)
                        if (!g.io[q].is_store && g.io[q].cls == LT_CLS_FULL && dtype_size(g.io[q].dtype) == 4) four_byte = true;
                    const bool integer_heavy = specialised(L) ? jit_integer_heavy(*L.jit_program) : lt_compiled_prefers_staging(L.compiled) == 0;
                    // Rows of 4097 to 8192 columns of a program with column vectors would need eight chunks per thread here
                    // (the vectors re-read for every row, two CTAs per SM): two CTAs of a cluster with four chunks per thread
                    // hold such a row instead (lt_c_rowc, as for rows beyond 8192 columns).
                    if (!specialised(L) && c->opt.cluster != 1 && g.n_pro > 0 && !integer_heavy && P.cpr > 512u) {
                        unsigned k = 0;
                        int cu = 0;
                        if (cluster_shape(P.cpr, true, c->opt.cluster, 0, &k, &cu)) {
                            const size_t cstage = lt_compiled_row_stage_bytes(L.compiled, cu);
                            unsigned cdepth = c->opt.compiled_depth >= 0 ? (unsigned)c->opt.compiled_depth : (four_byte ? 0u : 2u);
                            while (cdepth > 0 && cdepth * cstage > 72u * 1024u) --cdepth;
                            if (cstage == 0) cdepth = 0;
                            if (L.cluster_max < 0) {
                                int n = 0;
                                if (lt_compiled_cluster_occupancy(L.compiled, cu, 0, k, cdepth, &n) != cudaSuccess) {
                                    cudaGetLastError();
                                    n = 0;
                                }
                                L.cluster_max = n;
                            }
                            if (L.cluster_max >= 1) {
                                const unsigned clusters = (unsigned)std::min<uint64_t>(P.rows, (uint64_t)L.cluster_max);
                                if (ev0) cudaEventRecord(ev0, c->stream);
                                e = lt_compiled_launch_cluster(L.compiled, &P, cu, 0, clusters, k, cdepth, (uint64_t)c->wait_limit_ns, c->stream);
                                if (ev1) cudaEventRecord(ev1, c->stream);
                                c->status_pending = true;
                                done = true;
                            }
                        }
                    }
                    if (!done) {
                    int u = row_chunks_per_thread(P.cpr, g.n_pro > 0 && !integer_heavy, four_byte);
                    if (c->opt.compiled_row_u > 0 && !specialised(L)) u = (int)c->opt.compiled_row_u;
                    while (u < 8 && P.cpr > 128u * u) u *= 2;  // a row's group is at most one CTA of 128 threads
                    unsigned grp = 1, lg = 0;
                    while (grp * u < P.cpr) grp <<= 1, ++lg;
                    const unsigned threads = grp > 128 ? grp : 128;
                    // pipeline depth: stages of the next blocks' inputs in shared memory, within ~72 KB per CTA
                    const size_t stage = specialised(L) ? jit_row_stage_bytes(*L.jit_program, u, 128) : lt_compiled_row_stage_bytes(L.compiled, u);
                    // (not for programs bound by integer issue, nor for 4-byte inputs, which measured faster loaded directly:
                    // softmax f32 at 2048 columns 169 against 248 us)
                    const bool wants_ring = !integer_heavy && !four_byte;
                    unsigned depth = c->opt.compiled_depth >= 0 ? (unsigned)c->opt.compiled_depth : (wants_ring ? 2u : 0u);
                    while (depth > 0 && depth * stage > 72u * 1024u) --depth;
                    if (stage == 0 || threads != 128 || depth < 2) depth = 0;
                    const int occ = compiled_blocks(c, L, u, (int)threads, depth * stage);
                    const uint64_t blocks = ((uint64_t)P.rows + threads / grp - 1) / (threads / grp);
                    // one wave of persistent CTAs; with many blocks of rows per CTA, four waves balance the tail
                    // better (measured on [32768 x 2048])
                    const uint64_t resident = (uint64_t)c->sm_count * occ;
                    const unsigned rwaves = c->opt.waves > 0 ? waves : (blocks >= 16 * resident ? 4u : 1u);
                    unsigned grid = (unsigned)std::min<uint64_t>(blocks, resident * rwaves);
                    if (grid < 1) grid = 1;
                    if (ev0) cudaEventRecord(ev0, c->stream);
                    e = fast_launch(c, L, &P, u, grid, threads, grp, lg, depth, depth * stage);
                    if (ev1) cudaEventRecord(ev1, c->stream);
                    done = true;
                    }
                }
                if (done) c->stats.launches_compiled++;
            }
            if (done) {
                if (L.kind == K_EW) c->stats.launches_elementwise++;
                else c->stats.launches_row++;
            } else if (L.kind == K_EW) {
                if (!dry) {
                    uint64_t need = (P.n_chunks + LT_EW_THREADS - 1) / LT_EW_THREADS;
                    uint64_t want = std::min<uint64_t>(need, (uint64_t)c->sm_count * c->occ_ew * waves);
                    if (g.n_pro && P.rowcol && want < need) {
                        // loop-invariant column loads: a thread must stay on one column range, i.e. the chunk
                        // stride (grid x 256) must be a multiple of the chunks per row
                        uint64_t a = P.cpr, b = LT_EW_THREADS;
                        while (b) { uint64_t t = a % b; a = b; b = t; }
                        const uint64_t m = P.cpr / a;
                        want = (want + m - 1) / m * m;
                        if (want > need) want = need;  // one chunk per thread: nothing to keep invariant
                    }
                    unsigned grid = (unsigned)want;
                    if (grid < 1) grid = 1;
                    if (ev0) cudaEventRecord(ev0, c->stream);
                    e = lt_launch_ew(P, L.flavour, grid, c->stream);
                    if (ev1) cudaEventRecord(ev1, c->stream);
                }
                c->stats.launches_elementwise++;
            } else {
                if (!dry) {
                    uint64_t blocks = ((uint64_t)P.rows + P.rows_per_cta - 1) / P.rows_per_cta;
                    unsigned per_sm = (unsigned)std::max(1, c->occ_row * 256 / (int)L.threads);
                    unsigned grid = (unsigned)std::min<uint64_t>(blocks, (uint64_t)c->sm_count * per_sm * waves);
                    if (grid < 1) grid = 1;
                    if (ev0) cudaEventRecord(ev0, c->stream);
                    e = lt_launch_row(P, L.flavour, grid, L.threads, c->stream);
                    if (ev1) cudaEventRecord(ev1, c->stream);
                }
                c->stats.launches_row++;
            }
        }
        if (ev0) c->timed.push_back(TimedLaunch{ev0, ev1, (uint8_t)(L.kind == K_RED ? K_ROW : L.kind == K_VIEW ? K_EW : L.kind), L.bytes});
        if (e != cudaSuccess) {
            release_all(true);
            return fail(c, LT_ERR_CUDA, std::string("kernel launch: ") + cudaGetErrorString(e));
        }
        c->stats.kernels_launched++;
        c->stats.bytes_planned += L.bytes;
    }
    release_all(false);  // stream-ordered: later users of this memory queue behind the kernels above
    c->stats.outputs_donated += donated;
    c->stats.outputs_allocated += allocated;
    c->stats.temporaries_allocated += plan.temp_bytes.size();
    return LT_OK;
}

}  // namespace lt
