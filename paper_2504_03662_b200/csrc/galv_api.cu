// C boundary of libgalv.so: argument checks, workspace carve-up, launches.
// Every entry point is declared and documented in include/galv.h.

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "galv_internal.h"

// Built with -DGALV_NVTX (python -m paper_2504_03662_b200.build --nvtx), the three calls of the path open a named
// range each, so that a timeline profiler shows cost model / search / plan step; the default build has no such
// dependency.
#ifdef GALV_NVTX
#include <nvtx3/nvToolsExt.h>
struct GalvRange {
    explicit GalvRange(const char* name) { nvtxRangePushA(name); }
    ~GalvRange() { nvtxRangePop(); }
};
#define GALV_RANGE(name) GalvRange galv_range_(name)
#else
#define GALV_RANGE(name) do { } while (0)
#endif

namespace {

void set_err(galv_ctx* ctx, const char* fmt, const char* detail = "")
{
    if (ctx) std::snprintf(ctx->err, sizeof(ctx->err), fmt, detail);
}

int cuda_fail(galv_ctx* ctx, const char* where, cudaError_t e)
{
    if (ctx) std::snprintf(ctx->err, sizeof(ctx->err), "%s: %s", where, cudaGetErrorString(e));
    return GALV_ERR_CUDA;
}

bool shape_ok(const galv_shape* sh)
{
    return sh && sh->B >= 1 && sh->S >= 1 && sh->S <= 256 && sh->Lmax >= 1 && sh->Lmax <= 65535 && sh->M >= 0 &&
           sh->M < (1 << 24) && sh->m_pitch >= sh->M + 1 && (sh->m_pitch % 32) == 0;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

// Device arena of galv_search_host.
struct Arena { size_t L, layers, strat, inst, time_q, mem_q, trans_q, C, A, C_last, opt, plan, used, status, ws, total; };

Arena arena_layout(const galv_shape* sh, bool with_model)
{
    Arena a;
    const size_t B = sh->B, Lm = sh->Lmax, S = sh->S, P = sh->m_pitch;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align256(off + bytes); return o; };
    a.L = take(B * 4);
    a.layers = take(with_model ? B * Lm * sizeof(galv_layer_desc) : 0);
    a.strat = take(with_model ? S * sizeof(galv_strategy_desc) : 0);
    a.inst = take(with_model ? B * sizeof(galv_inst_params) : 0);
    a.time_q = take(B * Lm * S * 4);
    a.mem_q = take(B * Lm * S * 4);
    a.trans_q = take(B * S * S * 4 * ((sh->flags & GALV_TRANS_PER_LAYER) ? Lm : 1));
    a.C = take((sh->flags & GALV_STORE_C_FULL) ? B * Lm * S * P * 4 : 0);
    a.A = take((sh->flags & GALV_STORE_ARGMIN) ? B * Lm * S * P : 0);
    a.C_last = take(B * S * P * 4);
    a.opt = take(B * 4);
    a.plan = take(B * Lm * 4);
    a.used = take(B * 4);
    a.status = take(B * 4);
    a.ws = take(galv_ws_layout(sh).total);
    a.total = off;
    return a;
}

}  // namespace

int galv_set_error(galv_ctx* ctx, int code, const char* text)
{
    if (ctx) std::snprintf(ctx->err, sizeof(ctx->err), "%s", text);
    return code;
}

extern "C" {

int galv_create(galv_ctx** out, int device_ordinal)
{
    if (!out) return GALV_ERR_INVALID_ARG;
    *out = nullptr;
    cudaDeviceProp prop;
    cudaError_t e = cudaGetDeviceProperties(&prop, device_ordinal);
    if (e != cudaSuccess) { cudaGetLastError(); return GALV_ERR_CUDA; }   // clear the non-sticky error
    if (prop.major != 10) return GALV_ERR_UNSUPPORTED;
    galv_ctx* ctx = new (std::nothrow) galv_ctx;
    if (!ctx) return GALV_ERR_CUDA;
    ctx->device = device_ordinal;
    ctx->num_sms = prop.multiProcessorCount;
    ctx->smem_optin = (int)prop.sharedMemPerBlockOptin;
    ctx->err[0] = 0;
    ctx->profiling = 0;
    ctx->prof_count = 0;
    for (auto& ev : ctx->pev) ev = nullptr;
    int cur = -1;
    cudaGetDevice(&cur);
    if (cur != device_ordinal) cudaSetDevice(device_ordinal);
    e = galv_dp_configure(ctx);
    if (e == cudaSuccess) e = galv_cluster_configure(ctx);
    for (auto& ev : ctx->pev)
        if (e == cudaSuccess) e = cudaEventCreate(&ev);
    if (cur >= 0 && cur != device_ordinal) cudaSetDevice(cur);
    if (e != cudaSuccess) {
        for (auto& ev : ctx->pev)
            if (ev) cudaEventDestroy(ev);
        delete ctx;
        return GALV_ERR_CUDA;
    }
    *out = ctx;
    return GALV_OK;
}

int galv_destroy(galv_ctx* ctx)
{
    if (ctx)
        for (auto& ev : ctx->pev)
            if (ev) cudaEventDestroy(ev);
    delete ctx;
    return GALV_OK;
}

const char* galv_strerror(int code)
{
    switch (code) {
    case GALV_OK: return "ok";
    case GALV_ERR_INVALID_ARG: return "invalid argument";
    case GALV_ERR_UNSUPPORTED: return "unsupported device (needs compute capability 10.x)";
    case GALV_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case GALV_ERR_CUDA: return "CUDA call failed";
    case GALV_ERR_TIMEOUT: return "bounded device-side wait ran out";
    default: return "unknown error code";
    }
}

const char* galv_last_error(const galv_ctx* ctx) { return ctx ? ctx->err : "no context"; }

int galv_eval_costs(galv_ctx* ctx, const galv_shape* sh, const int32_t* L, const galv_layer_desc* layers,
                    int64_t layer_stride_B, const galv_strategy_desc* strat, const galv_inst_params* inst,
                    double* time_s, double* mem_bytes, int32_t* time_q, int32_t* mem_q, int32_t* trans_q,
                    int32_t* status, void* stream)
{
    GALV_RANGE("galv_eval_costs");
    if (!ctx) return GALV_ERR_INVALID_ARG;
    if (!shape_ok(sh)) { set_err(ctx, "galv_eval_costs: shape outside limits"); return GALV_ERR_INVALID_ARG; }
    if (!L || !layers || !strat || !inst || !time_q || !mem_q || !trans_q || !status) {
        set_err(ctx, "galv_eval_costs: NULL required pointer");
        return GALV_ERR_INVALID_ARG;
    }
    if (layer_stride_B != 0 && layer_stride_B < sh->Lmax) {
        set_err(ctx, "galv_eval_costs: layer_stride_B must be 0 or >= Lmax");
        return GALV_ERR_INVALID_ARG;
    }
    if (sh->flags & GALV_TRANS_PER_LAYER) {
        set_err(ctx, "galv_eval_costs: the cost model writes one transition matrix per instance (no GALV_TRANS_PER_LAYER)");
        return GALV_ERR_INVALID_ARG;
    }
    cudaError_t e = galv_costs_launch(sh, L, layers, layer_stride_B, strat, inst, time_s, mem_bytes, time_q, mem_q,
                                      trans_q, status, (cudaStream_t)stream);
    return e == cudaSuccess ? GALV_OK : cuda_fail(ctx, "galv_eval_costs", e);
}

size_t galv_dp_workspace_bytes(const galv_ctx* ctx, const galv_shape* sh)
{
    (void)ctx;
    if (!shape_ok(sh)) return 0;
    return galv_ws_layout(sh).total;
}

int galv_dp_search(galv_ctx* ctx, const galv_shape* sh, const int32_t* L, const int32_t* time_q,
                   const int32_t* mem_q, const int32_t* trans_q, int32_t* C, uint8_t* A, int32_t* C_last,
                   void* workspace, size_t workspace_bytes, int32_t* status, void* stream)
{
    GALV_RANGE("galv_dp_search");
    if (!ctx) return GALV_ERR_INVALID_ARG;
    if (!shape_ok(sh)) { set_err(ctx, "galv_dp_search: shape outside limits"); return GALV_ERR_INVALID_ARG; }
    if (!L || !time_q || !mem_q || !trans_q || !C_last || !status) {
        set_err(ctx, "galv_dp_search: NULL required pointer");
        return GALV_ERR_INVALID_ARG;
    }
    const bool full = (sh->flags & GALV_STORE_C_FULL) != 0, argm = (sh->flags & GALV_STORE_ARGMIN) != 0;
    if (full != (C != nullptr) || argm != (A != nullptr)) {
        set_err(ctx, "galv_dp_search: C / A must be given exactly when GALV_STORE_C_FULL / GALV_STORE_ARGMIN is set");
        return GALV_ERR_INVALID_ARG;
    }
    if (!aligned16(C) || !aligned16(C_last) || !aligned16(trans_q)) {
        set_err(ctx, "galv_dp_search: tables must be 16-byte aligned");
        return GALV_ERR_INVALID_ARG;
    }
    const WsLayout w = galv_ws_layout(sh);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < w.total) {
        set_err(ctx, "galv_dp_search: workspace missing, not 256-byte aligned, or smaller than galv_dp_workspace_bytes");
        return GALV_ERR_WORKSPACE;
    }
    char* ws = static_cast<char*>(workspace);
    DpArgs a;
    a.B = sh->B; a.Lmax = sh->Lmax; a.S = sh->S; a.M = sh->M; a.m_pitch = sh->m_pitch;
    a.L = L; a.time_q = time_q; a.mem_q = mem_q; a.trans_q = trans_q;
    a.trans_inst = galv_trans_inst(sh); a.trans_layer = galv_trans_layer(sh);
    a.C = C; a.A = A; a.C_last = C_last;
    a.roll = reinterpret_cast<int32_t*>(ws + w.roll);
    a.order = reinterpret_cast<int32_t*>(ws + w.order);
    a.nactive = reinterpret_cast<int32_t*>(ws + w.nactive);
    a.scratch = reinterpret_cast<int32_t*>(ws + w.scratch);
    a.work = reinterpret_cast<unsigned long long*>(a.scratch + 2 * (sh->Lmax + 2));
    a.istart = reinterpret_cast<long long*>(ws + w.istart);
    a.tcount = reinterpret_cast<int32_t*>(ws + w.tcount);
    a.trans_p = reinterpret_cast<uint32_t*>(ws + w.trans_p);
    a.trans_k = reinterpret_cast<int32_t*>(ws + w.trans_p);
    a.keyed = 0;
    a.err = reinterpret_cast<int32_t*>(ws + w.err);
    a.tile_done = reinterpret_cast<int32_t*>(ws + w.tile_done);
    a.maxmem = a.err + 1;
    a.minmem_l = reinterpret_cast<int32_t*>(ws + w.minmem_l);
    a.ntiles = reinterpret_cast<int32_t*>(ws + w.ntiles);
    a.front = reinterpret_cast<int32_t*>(ws + w.front);
    a.status = status;
    a.withhold = 0;
    cudaError_t e = galv_dp_launch(ctx, sh, a, (cudaStream_t)stream);
    return e == cudaSuccess ? GALV_OK : cuda_fail(ctx, "galv_dp_search", e);
}

int galv_dp_search_path(galv_ctx* ctx, const galv_shape* sh, const void* workspace, int32_t* packed, void* stream)
{
    if (!ctx) return GALV_ERR_INVALID_ARG;
    if (!shape_ok(sh) || !workspace || !packed) { set_err(ctx, "galv_dp_search_path: bad shape or NULL pointer"); return GALV_ERR_INVALID_ARG; }
    const WsLayout w = galv_ws_layout(sh);
    int32_t flags[4] = {0, 0, 0, 0};                       // error flag, largest mem, largest trans, path
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaMemcpy(flags, static_cast<const char*>(workspace) + w.err, sizeof(flags), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(ctx, "galv_dp_search_path", e);
    *packed = flags[3];
    return GALV_OK;
}

int galv_backtrack(galv_ctx* ctx, const galv_shape* sh, const int32_t* L, const int32_t* time_q,
                   const int32_t* mem_q, const int32_t* trans_q, const int32_t* C, const uint8_t* A,
                   const int32_t* C_last, const int32_t* budget, int32_t* opt_cost, int32_t* plan,
                   int32_t* mem_used, int32_t* status, void* stream)
{
    GALV_RANGE("galv_backtrack");
    if (!ctx) return GALV_ERR_INVALID_ARG;
    if (!shape_ok(sh)) { set_err(ctx, "galv_backtrack: shape outside limits"); return GALV_ERR_INVALID_ARG; }
    if (!L || !time_q || !mem_q || !trans_q || !C_last || !opt_cost || !status) {
        set_err(ctx, "galv_backtrack: NULL required pointer");
        return GALV_ERR_INVALID_ARG;
    }
    if (plan && !A && !C) {
        set_err(ctx, "galv_backtrack: a plan needs the argmin table A or the full table C");
        return GALV_ERR_INVALID_ARG;
    }
    cudaError_t e = galv_backtrack_launch(sh, L, time_q, mem_q, trans_q, C, A, C_last, budget, opt_cost, plan,
                                          mem_used, status, (cudaStream_t)stream);
    return e == cudaSuccess ? GALV_OK : cuda_fail(ctx, "galv_backtrack", e);
}

size_t galv_search_host_arena_bytes(const galv_ctx* ctx, const galv_shape* sh, int with_model)
{
    (void)ctx;
    if (!shape_ok(sh)) return 0;
    return arena_layout(sh, with_model != 0).total;
}

int galv_search_host(galv_ctx* ctx, const galv_shape* sh, const int32_t* L, const galv_layer_desc* layers,
                     int64_t layer_stride_B, const galv_strategy_desc* strat, const galv_inst_params* inst,
                     const int32_t* time_q, const int32_t* mem_q, const int32_t* trans_q, int32_t* opt_cost,
                     int32_t* plan, int32_t* mem_used, int32_t* status, void* arena, size_t arena_bytes,
                     void* stream)
{
    if (!ctx) return GALV_ERR_INVALID_ARG;
    if (!shape_ok(sh)) { set_err(ctx, "galv_search_host: shape outside limits"); return GALV_ERR_INVALID_ARG; }
    const bool model = layers != nullptr;
    if (!L || !opt_cost || !plan || !mem_used || !status || (model && (!strat || !inst)) ||
        (!model && (!time_q || !mem_q || !trans_q))) {
        set_err(ctx, "galv_search_host: NULL required pointer");
        return GALV_ERR_INVALID_ARG;
    }
    if (!(sh->flags & (GALV_STORE_C_FULL | GALV_STORE_ARGMIN))) {
        set_err(ctx, "galv_search_host: flags must keep C or A so that a plan can be produced");
        return GALV_ERR_INVALID_ARG;
    }
    const Arena ar = arena_layout(sh, model);
    if (!arena || (reinterpret_cast<uintptr_t>(arena) & 255) || arena_bytes < ar.total) {
        set_err(ctx, "galv_search_host: arena missing, not 256-byte aligned, or smaller than galv_search_host_arena_bytes");
        return GALV_ERR_WORKSPACE;
    }
    cudaStream_t st = (cudaStream_t)stream;
    char* d = static_cast<char*>(arena);
    const size_t B = sh->B, Lm = sh->Lmax, S = sh->S;
    cudaError_t e;
#define GALV_H2D(dst_off, src, bytes)                                                              \
    if ((e = cudaMemcpyAsync(d + (dst_off), (src), (bytes), cudaMemcpyHostToDevice, st)) != cudaSuccess) \
        return cuda_fail(ctx, "galv_search_host (copy in)", e)
    GALV_H2D(ar.L, L, B * 4);
    int32_t* d_tq = reinterpret_cast<int32_t*>(d + ar.time_q);
    int32_t* d_mq = reinterpret_cast<int32_t*>(d + ar.mem_q);
    int32_t* d_xq = reinterpret_cast<int32_t*>(d + ar.trans_q);
    int32_t* d_status = reinterpret_cast<int32_t*>(d + ar.status);
    const int32_t* d_L = reinterpret_cast<const int32_t*>(d + ar.L);
    int rc;
    if (model) {
        const size_t rows = layer_stride_B == 0 ? Lm : B * (size_t)layer_stride_B;
        if (layer_stride_B != 0 && layer_stride_B != (int64_t)Lm) {
            set_err(ctx, "galv_search_host: layer_stride_B must be 0 or Lmax");
            return GALV_ERR_INVALID_ARG;
        }
        GALV_H2D(ar.layers, layers, rows * sizeof(galv_layer_desc));
        GALV_H2D(ar.strat, strat, S * sizeof(galv_strategy_desc));
        GALV_H2D(ar.inst, inst, B * sizeof(galv_inst_params));
        rc = galv_eval_costs(ctx, sh, d_L, reinterpret_cast<const galv_layer_desc*>(d + ar.layers), layer_stride_B,
                             reinterpret_cast<const galv_strategy_desc*>(d + ar.strat),
                             reinterpret_cast<const galv_inst_params*>(d + ar.inst), nullptr, nullptr, d_tq, d_mq, d_xq,
                             d_status, stream);
        if (rc != GALV_OK) return rc;
    } else {
        GALV_H2D(ar.time_q, time_q, B * Lm * S * 4);
        GALV_H2D(ar.mem_q, mem_q, B * Lm * S * 4);
        GALV_H2D(ar.trans_q, trans_q, B * S * S * 4 * ((sh->flags & GALV_TRANS_PER_LAYER) ? Lm : 1));
    }
#undef GALV_H2D
    int32_t* d_C = (sh->flags & GALV_STORE_C_FULL) ? reinterpret_cast<int32_t*>(d + ar.C) : nullptr;
    uint8_t* d_A = (sh->flags & GALV_STORE_ARGMIN) ? reinterpret_cast<uint8_t*>(d + ar.A) : nullptr;
    int32_t* d_last = reinterpret_cast<int32_t*>(d + ar.C_last);
    rc = galv_dp_search(ctx, sh, d_L, d_tq, d_mq, d_xq, d_C, d_A, d_last, d + ar.ws, ar.total - ar.ws, d_status, stream);
    if (rc != GALV_OK) return rc;
    rc = galv_backtrack(ctx, sh, d_L, d_tq, d_mq, d_xq, d_C, d_A, d_last, nullptr,
                        reinterpret_cast<int32_t*>(d + ar.opt), reinterpret_cast<int32_t*>(d + ar.plan),
                        reinterpret_cast<int32_t*>(d + ar.used), d_status, stream);
    if (rc != GALV_OK) return rc;
#define GALV_D2H(dst, src_off, bytes)                                                              \
    if ((e = cudaMemcpyAsync((dst), d + (src_off), (bytes), cudaMemcpyDeviceToHost, st)) != cudaSuccess) \
        return cuda_fail(ctx, "galv_search_host (copy out)", e)
    GALV_D2H(opt_cost, ar.opt, B * 4);
    GALV_D2H(plan, ar.plan, B * Lm * 4);
    GALV_D2H(mem_used, ar.used, B * 4);
    GALV_D2H(status, ar.status, B * 4);
#undef GALV_D2H
    if ((e = cudaStreamSynchronize(st)) != cudaSuccess) return cuda_fail(ctx, "galv_search_host (sync)", e);
    for (size_t i = 0; i < B; ++i)
        if (status[i] & GALV_STATUS_TIMEOUT) { set_err(ctx, "galv_search_host: device-side wait ran out"); return GALV_ERR_TIMEOUT; }
    return GALV_OK;
}

int galv_set_profiling(galv_ctx* ctx, int on)
{
    if (!ctx) return GALV_ERR_INVALID_ARG;
    ctx->profiling = on != 0;
    ctx->prof_count = 0;
    return GALV_OK;
}

int galv_last_layer_loop_ms(galv_ctx* ctx, float* ms)
{
    if (!ctx || !ms) return GALV_ERR_INVALID_ARG;
    if (ctx->prof_count < 1) { set_err(ctx, "galv_last_layer_loop_ms: no profiled search yet"); return GALV_ERR_INVALID_ARG; }
    const int k = (ctx->prof_count - 1) % 64;
    cudaError_t e = cudaEventSynchronize(ctx->pev[2 * k + 1]);
    if (e == cudaSuccess) e = cudaEventElapsedTime(ms, ctx->pev[2 * k], ctx->pev[2 * k + 1]);
    return e == cudaSuccess ? GALV_OK : cuda_fail(ctx, "galv_last_layer_loop_ms", e);
}

int galv_layer_loop_ms_stats(galv_ctx* ctx, float* mean_ms, float* min_ms, float* max_ms, int* searches)
{
    if (!ctx || !mean_ms || !min_ms || !max_ms || !searches) return GALV_ERR_INVALID_ARG;
    if (ctx->prof_count < 1) { set_err(ctx, "galv_layer_loop_ms_stats: no profiled search yet"); return GALV_ERR_INVALID_ARG; }
    const int n = ctx->prof_count < 64 ? ctx->prof_count : 64;
    double sum = 0.0;
    float lo = 0.f, hi = 0.f;
    for (int j = 0; j < n; ++j) {
        const int k = (ctx->prof_count - 1 - j) % 64;
        float ms = 0.f;
        cudaError_t e = cudaEventSynchronize(ctx->pev[2 * k + 1]);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, ctx->pev[2 * k], ctx->pev[2 * k + 1]);
        if (e != cudaSuccess) return cuda_fail(ctx, "galv_layer_loop_ms_stats", e);
        sum += ms;
        if (j == 0 || ms < lo) lo = ms;
        if (j == 0 || ms > hi) hi = ms;
    }
    *mean_ms = (float)(sum / n); *min_ms = lo; *max_ms = hi; *searches = n;
    return GALV_OK;
}

int galv_probe_int_alu(galv_ctx* ctx, int kind, int iters, double* ops_per_s, void* stream)
{
    if (!ctx || !ops_per_s || iters < 1 || kind < 0 || kind > 4) return GALV_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    cudaEvent_t e0, e1;
    cudaError_t e;
    if ((e = cudaEventCreate(&e0)) != cudaSuccess) return cuda_fail(ctx, "galv_probe_int_alu", e);
    if ((e = cudaEventCreate(&e1)) != cudaSuccess) { cudaEventDestroy(e0); return cuda_fail(ctx, "galv_probe_int_alu", e); }
    long long ops = 0;
    float best = 1e30f;
    e = galv_probe_launch(ctx, kind, iters, nullptr, st, &ops);            // warm-up
    for (int rep = 0; rep < 5 && e == cudaSuccess; ++rep) {
        cudaEventRecord(e0, st);
        e = galv_probe_launch(ctx, kind, iters, nullptr, st, &ops);
        cudaEventRecord(e1, st);
        if (e == cudaSuccess) e = cudaEventSynchronize(e1);
        float ms = 0.f;
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
        if (e == cudaSuccess && ms < best) best = ms;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (e != cudaSuccess) return cuda_fail(ctx, "galv_probe_int_alu", e);
    *ops_per_s = (double)ops / ((double)best * 1e-3);
    return GALV_OK;
}

}  // extern "C"
