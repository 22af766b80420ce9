// Stage partitioning on top of the layer-wise search.
//
// (Sections 2 and 3 of the paper: layers are spread over pipeline stages so that the stages are
// balanced, and re-cut when one becomes the bottleneck.)  The batch is built with one instance per
// start layer a (its layers are a, a+1, ...); the search's table then holds, at layer n-1 and the
// full budget, the optimum of the stage made of layers a .. a+n-1.  layer_optima_kernel reads those
// optima out; stage_partition_kernel cuts the model into P stages minimising the slowest stage:
//   f[1][b] = opt(0,b),   f[k][b] = min_{k-1 <= a < b} max( f[k-1][a], opt(a,b) ).
// P * Lm^2 comparisons (a few million at most): one CTA, threads over b, tables in shared memory.

#include "galv_internal.h"

namespace {

constexpr int kInf = GALV_INF;

// opt_l[i][l] = min_s C[i][l][s][budget_i] for l < L[i]; GALV_INF beyond and for flagged instances.
__global__ void layer_optima_kernel(int B, int Lmax, int S, int M, int m_pitch, const int32_t* __restrict__ L,
                                    const int32_t* __restrict__ C, const int32_t* __restrict__ budget,
                                    const int32_t* __restrict__ status, int32_t* __restrict__ opt_l)
{
    const int lane = threadIdx.x & 31;
    const long long w = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (w >= (long long)B * Lmax) return;
    const int i = (int)(w / Lmax), l = (int)(w - (long long)i * Lmax);
    int best = kInf;
    const int bud = budget ? budget[i] : M;
    const bool ok = (status[i] & (GALV_STATUS_BAD_INPUT | GALV_STATUS_OVERFLOW_RISK | GALV_STATUS_TIMEOUT)) == 0 && l < L[i] && bud >= 0 && bud <= M;
    if (ok)
        for (int s = lane; s < S; s += 32) best = min(best, C[(((size_t)i * Lmax + l) * S + s) * m_pitch + bud]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) best = min(best, __shfl_xor_sync(0xffffffffu, best, o));
    if (lane == 0) opt_l[w] = best;
}

// f and g (argmin) are [P+1][Lm+1] ints in dynamic shared memory.
__global__ void stage_partition_kernel(int Lm, int P, const int32_t* __restrict__ range_opt, int32_t* __restrict__ cuts,
                                       int32_t* __restrict__ bottleneck)
{
    extern __shared__ int32_t sm[];
    int32_t* f = sm;
    int32_t* g = sm + (size_t)(P + 1) * (Lm + 1);
    const int W = Lm + 1;
    for (int k = 1; k <= P; ++k) {
        for (int b = threadIdx.x; b <= Lm; b += blockDim.x) {
            int best = kInf, arg = -1;
            if (b >= k) {
                if (k == 1) { best = range_opt[b - 1]; arg = 0; }
                else
                    for (int a = k - 1; a < b; ++a) {
                        const int v = max(f[(k - 1) * W + a], range_opt[(size_t)a * Lm + (b - a - 1)]);
                        if (v < best) { best = v; arg = a; }          // strict: the lowest a wins ties
                    }
            }
            if (best >= kInf) { best = kInf; arg = -1; }
            f[k * W + b] = best;
            g[k * W + b] = arg;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const int bn = f[P * W + Lm];
        *bottleneck = bn;
        if (bn < kInf) {
            int b = Lm;
            for (int k = P; k >= 1; --k) { cuts[k] = b; b = g[k * W + b]; }
            cuts[0] = 0;
        } else {
            for (int k = 0; k <= P; ++k) cuts[k] = -1;
        }
    }
}

}  // namespace

extern "C" {

int galv_layer_optima(galv_ctx* ctx, const galv_shape* sh, const int32_t* L, const int32_t* C, const int32_t* budget,
                      const int32_t* status, int32_t* opt_l, void* stream)
{
    if (!ctx) return GALV_ERR_INVALID_ARG;
    if (!sh || sh->B < 1 || sh->S < 1 || sh->Lmax < 1 || sh->M < 0 || sh->m_pitch < sh->M + 1 || !L || !C || !status || !opt_l)
        return galv_set_error(ctx, GALV_ERR_INVALID_ARG, "galv_layer_optima: bad shape or NULL pointer (needs the full table C)");
    const long long warps = (long long)sh->B * sh->Lmax;
    layer_optima_kernel<<<(unsigned)((warps + 3) / 4), 128, 0, (cudaStream_t)stream>>>(sh->B, sh->Lmax, sh->S, sh->M, sh->m_pitch,
                                                                                       L, C, budget, status, opt_l);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? GALV_OK : galv_set_error(ctx, GALV_ERR_CUDA, cudaGetErrorString(e));
}

int galv_stage_partition(galv_ctx* ctx, int32_t Lm, int32_t P, const int32_t* range_opt, int32_t* cuts,
                         int32_t* bottleneck, void* stream)
{
    if (!ctx) return GALV_ERR_INVALID_ARG;
    if (Lm < 1 || P < 1 || !range_opt || !cuts || !bottleneck)
        return galv_set_error(ctx, GALV_ERR_INVALID_ARG, "galv_stage_partition: Lm, P >= 1 and no NULL pointer");
    const size_t bytes = (size_t)2 * (P + 1) * (Lm + 1) * sizeof(int32_t);
    if (bytes > (size_t)ctx->smem_optin)
        return galv_set_error(ctx, GALV_ERR_INVALID_ARG, "galv_stage_partition: (P+1)*(Lm+1) tables exceed the shared memory of one CTA");
    cudaError_t e = cudaFuncSetAttribute(stage_partition_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess) {
        stage_partition_kernel<<<1, 256, bytes, (cudaStream_t)stream>>>(Lm, P, range_opt, cuts, bottleneck);
        e = cudaGetLastError();
    }
    return e == cudaSuccess ? GALV_OK : galv_set_error(ctx, GALV_ERR_CUDA, cudaGetErrorString(e));
}

}  // extern "C"
