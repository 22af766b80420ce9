// Re-search pipeline: cost model -> search -> plan, captured once in a CUDA graph and replayed.
//
// (Sections 3 and 4 of the paper: during training the selector re-evaluates the plan at intervals
// from fresh measurements.)  The descriptor tables stay in device memory; the caller overwrites the
// per-instance parameters (measured FLOP rate, link bandwidth, micro-batch) in place and replays
// the graph: one host call per re-search instead of a dozen launches.
// Also here: the cost and memory of a GIVEN plan under the current tables (what the running plan
// costs now), the other half of a switch decision.

#include <new>

#include "galv_internal.h"

struct galv_graph {
    cudaGraph_t graph;
    cudaGraphExec_t exec;
};

namespace {

// One warp per instance: cost(p) = sum_l time(l,p_l) + sum_{l>=1} trans(p_{l-1},p_l), mem = sum_l mem(l,p_l).
// -1 for both when the plan has an entry outside 0..S-1 within the instance's layers.
__global__ void plan_cost_kernel(int B, int Lmax, int S, long long trans_inst, long long trans_layer, const int32_t* __restrict__ L, const int32_t* __restrict__ time_q,
                                 const int32_t* __restrict__ mem_q, const int32_t* __restrict__ trans_q,
                                 const int32_t* __restrict__ plan, long long* __restrict__ cost, long long* __restrict__ mem_total)
{
    const int lane = threadIdx.x & 31;
    const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (i >= B) return;
    const int Li = L[i];
    long long c = 0, u = 0;
    int bad = (Li < 1 || Li > Lmax);
    if (!bad)
        for (int l = lane; l < Li; l += 32) {
            const int p = plan[(size_t)i * Lmax + l];
            if (p < 0 || p >= S) { bad = 1; continue; }
            c += time_q[((size_t)i * Lmax + l) * S + p];
            u += mem_q[((size_t)i * Lmax + l) * S + p];
            if (l >= 1) {
                const int q = plan[(size_t)i * Lmax + l - 1];
                if (q >= 0 && q < S) c += trans_q[(size_t)i * trans_inst + (size_t)l * trans_layer + (size_t)q * S + p];
            }
        }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        c += __shfl_xor_sync(0xffffffffu, c, o);
        u += __shfl_xor_sync(0xffffffffu, u, o);
        bad |= __shfl_xor_sync(0xffffffffu, bad, o);
    }
    if (lane == 0) {
        cost[i] = bad ? -1 : c;
        mem_total[i] = bad ? -1 : u;
    }
}

}  // namespace

extern "C" {

int galv_plan_cost(galv_ctx* ctx, const galv_shape* sh, const int32_t* L, const int32_t* time_q, const int32_t* mem_q,
                   const int32_t* trans_q, const int32_t* plan, int64_t* cost, int64_t* mem_total, void* stream)
{
    if (!ctx) return GALV_ERR_INVALID_ARG;
    if (!sh || sh->B < 1 || sh->S < 1 || sh->Lmax < 1 || !L || !time_q || !mem_q || !trans_q || !plan || !cost || !mem_total)
        return galv_set_error(ctx, GALV_ERR_INVALID_ARG, "galv_plan_cost: bad shape or NULL pointer");
    plan_cost_kernel<<<(sh->B + 3) / 4, 128, 0, (cudaStream_t)stream>>>(sh->B, sh->Lmax, sh->S, galv_trans_inst(sh), galv_trans_layer(sh), L, time_q, mem_q, trans_q, plan,
                                                                       reinterpret_cast<long long*>(cost),
                                                                       reinterpret_cast<long long*>(mem_total));
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? GALV_OK : galv_set_error(ctx, GALV_ERR_CUDA, cudaGetErrorString(e));
}

int galv_graph_create(galv_ctx* ctx, const galv_shape* sh, const int32_t* L, const galv_layer_desc* layers,
                      int64_t layer_stride_B, const galv_strategy_desc* strat, const galv_inst_params* inst,
                      int32_t* time_q, int32_t* mem_q, int32_t* trans_q, int32_t* C, uint8_t* A, int32_t* C_last,
                      void* workspace, size_t workspace_bytes, const int32_t* budget, int32_t* opt_cost, int32_t* plan,
                      int32_t* mem_used, int32_t* status, void* stream, galv_graph** out)
{
    if (!ctx || !out) return GALV_ERR_INVALID_ARG;
    *out = nullptr;
    cudaStream_t st = (cudaStream_t)stream;
    if (!st) return galv_set_error(ctx, GALV_ERR_INVALID_ARG, "galv_graph_create: capture needs a non-default stream");
    cudaError_t e = cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal);
    if (e != cudaSuccess) return galv_set_error(ctx, GALV_ERR_CUDA, cudaGetErrorString(e));
    int rc = GALV_OK;
    if (layers) rc = galv_eval_costs(ctx, sh, L, layers, layer_stride_B, strat, inst, nullptr, nullptr, time_q, mem_q, trans_q, status, stream);
    if (rc == GALV_OK) rc = galv_dp_search(ctx, sh, L, time_q, mem_q, trans_q, C, A, C_last, workspace, workspace_bytes, status, stream);
    if (rc == GALV_OK) rc = galv_backtrack(ctx, sh, L, time_q, mem_q, trans_q, C, A, C_last, budget, opt_cost, plan, mem_used, status, stream);
    cudaGraph_t g = nullptr;
    e = cudaStreamEndCapture(st, &g);                     // always end the capture, also after a failed call
    if (rc != GALV_OK) { if (g) cudaGraphDestroy(g); return rc; }
    if (e != cudaSuccess || !g) return galv_set_error(ctx, GALV_ERR_CUDA, cudaGetErrorString(e));
    cudaGraphExec_t x = nullptr;
    e = cudaGraphInstantiate(&x, g, 0);
    if (e != cudaSuccess) { cudaGraphDestroy(g); return galv_set_error(ctx, GALV_ERR_CUDA, cudaGetErrorString(e)); }
    galv_graph* gg = new (std::nothrow) galv_graph;
    if (!gg) { cudaGraphExecDestroy(x); cudaGraphDestroy(g); return galv_set_error(ctx, GALV_ERR_CUDA, "out of host memory"); }
    gg->graph = g;
    gg->exec = x;
    *out = gg;
    return GALV_OK;
}

int galv_graph_launch(galv_ctx* ctx, galv_graph* g, void* stream)
{
    if (!ctx || !g) return GALV_ERR_INVALID_ARG;
    const cudaError_t e = cudaGraphLaunch(g->exec, (cudaStream_t)stream);
    return e == cudaSuccess ? GALV_OK : galv_set_error(ctx, GALV_ERR_CUDA, cudaGetErrorString(e));
}

int galv_graph_destroy(galv_graph* g)
{
    if (g) {
        cudaGraphExecDestroy(g->exec);
        cudaGraphDestroy(g->graph);
        delete g;
    }
    return GALV_OK;
}

}  // extern "C"
