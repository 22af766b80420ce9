// Plan switch: the cost of leaving the running plan, and the decision to leave it.
// (Sections 3 and 4 of the paper: during training the monitor re-evaluates, the optimiser proposes
// a plan and the manager reshards the job; the paper gives no rule for when that pays.)
// Moving layer l from its current strategy c to s reshards the layer once, priced by the cost
// model's transition entry trans_l(c, s); spread over `horizon` iterations it adds
// trans_l(c, s) / horizon to time(l, s).  The search then weighs iteration time against the price
// of getting there, and the job switches only when the new optimum beats staying by a margin.
// Both kernels are elementwise and launch-latency bound.

#include "galv_internal.h"

namespace {

__global__ void switch_cost_kernel(int B, int Lmax, int S, long long trans_inst, long long trans_layer,
                                   const int32_t* __restrict__ L, const int32_t* __restrict__ time_q,
                                   const int32_t* __restrict__ trans_q, const int32_t* __restrict__ cur_plan,
                                   const int32_t* __restrict__ horizon, int32_t* __restrict__ time_out)
{
    const long long n = (long long)B * Lmax * S;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
        const int s = (int)(e % S);
        const long long il = e / S;
        const int l = (int)(il % Lmax);
        const int i = (int)(il / Lmax);
        long long v = time_q[e];
        const int Li = L[i];
        if (Li >= 1 && Li <= Lmax && l < Li) {
            const int c = cur_plan[il];
            if (c >= 0 && c < S) {
                const long long h = horizon[i] < 1 ? 1 : horizon[i];
                v += (long long)trans_q[(long long)i * trans_inst + (long long)l * trans_layer + (long long)c * S + s] / h;
            }
        }
        time_out[e] = v >= GALV_INF ? GALV_INF : (int32_t)v;
    }
}

__global__ void switch_decision_kernel(int B, const long long* __restrict__ cur_cost, const int32_t* __restrict__ new_cost,
                                       const int32_t* __restrict__ new_status, int hysteresis_permille,
                                       int32_t* __restrict__ decision)
{
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < B; i += gridDim.x * blockDim.x) {
        const long long nw = new_cost[i], cur = cur_cost[i];
        int d;
        if (new_status[i] != 0 || nw >= GALV_INF || nw < 0) d = 0;           // nothing to switch to
        else if (cur < 0 || cur >= GALV_INF) d = 1;                          // the running plan no longer fits
        else d = nw * (1000 + (long long)hysteresis_permille) < cur * 1000;
        decision[i] = d;
    }
}

}  // namespace

extern "C" int galv_add_switch_cost(galv_ctx* ctx, const galv_shape* sh, const int32_t* L, const int32_t* time_q,
                                    const int32_t* trans_q, const int32_t* cur_plan, const int32_t* horizon,
                                    int32_t* time_out, void* stream)
{
    if (!ctx) return GALV_ERR_INVALID_ARG;
    if (!sh || sh->B < 1 || sh->Lmax < 1 || sh->S < 1 || sh->S > 256 || !L || !time_q || !trans_q || !cur_plan || !horizon || !time_out)
        return galv_set_error(ctx, GALV_ERR_INVALID_ARG, "galv_add_switch_cost: bad shape or NULL pointer");
    const long long n = (long long)sh->B * sh->Lmax * sh->S;
    long long blocks = (n + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    switch_cost_kernel<<<(int)blocks, 256, 0, (cudaStream_t)stream>>>(sh->B, sh->Lmax, sh->S, galv_trans_inst(sh), galv_trans_layer(sh),
                                                                      L, time_q, trans_q, cur_plan, horizon, time_out);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? GALV_OK : galv_set_error(ctx, GALV_ERR_CUDA, cudaGetErrorString(e));
}

extern "C" int galv_switch_decision(galv_ctx* ctx, int32_t B, const int64_t* cur_cost, const int32_t* new_cost,
                                    const int32_t* new_status, int32_t hysteresis_permille, int32_t* decision, void* stream)
{
    if (!ctx) return GALV_ERR_INVALID_ARG;
    if (B < 1 || !cur_cost || !new_cost || !new_status || !decision || hysteresis_permille < 0)
        return galv_set_error(ctx, GALV_ERR_INVALID_ARG, "galv_switch_decision: B >= 1, hysteresis >= 0 and no NULL pointer");
    const int blocks = (B + 255) / 256 > 1024 ? 1024 : (B + 255) / 256;
    switch_decision_kernel<<<blocks, 256, 0, (cudaStream_t)stream>>>(B, reinterpret_cast<const long long*>(cur_cost), new_cost, new_status,
                                                                     hysteresis_permille, decision);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? GALV_OK : galv_set_error(ctx, GALV_ERR_CUDA, cudaGetErrorString(e));
}
