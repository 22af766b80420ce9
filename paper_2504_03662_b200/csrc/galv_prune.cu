// Dominated-strategy prune before the search, and the table compaction / plan expansion around it.
// (Section 3 of the paper: candidates are pruned before the dynamic program runs.)
//
// Strategy s goes when another strategy d is at least as good in every layer of every instance
// (time, memory) and in every transition (row and column of trans), and either d < s or d is
// strictly faster everywhere: then the search result, plan included, is unchanged.
// One CTA per strategy s; it tries the dominators d one after the other, each test a block-wide
// AND over B*L + 2*B*S comparisons.  Microseconds of work; launch-latency bound.

#include "galv_internal.h"

namespace {

__global__ void prune_kernel(int B, int Lmax, int S, const int32_t* __restrict__ L, const int32_t* __restrict__ time_q,
                             const int32_t* __restrict__ mem_q, const int32_t* __restrict__ trans_q, int32_t* __restrict__ keep)
{
    const int s = blockIdx.x;
    __shared__ int s_dom, s_strict;
    const long long nlay = (long long)B * Lmax, ntr = (long long)B * S;
    int kept = 1;
    for (int d = 0; d < S && kept; ++d) {
        if (d == s) continue;
        __syncthreads();
        if (threadIdx.x == 0) { s_dom = 1; s_strict = 1; }
        __syncthreads();
        int dom = 1, strict = 1;
        for (long long e = threadIdx.x; e < nlay && dom; e += blockDim.x) {
            const int i = (int)(e / Lmax), l = (int)(e - (long long)i * Lmax);
            const int Li = L[i];
            if (Li < 1 || Li > Lmax || l >= Li) continue;
            const size_t o = ((size_t)i * Lmax + l) * S;
            const int ts = time_q[o + s], td = time_q[o + d];
            if (td > ts || mem_q[o + d] > mem_q[o + s]) dom = 0;
            if (td >= ts) strict = 0;
        }
        for (long long e = threadIdx.x; e < ntr && dom; e += blockDim.x) {
            const int i = (int)(e / S), k = (int)(e - (long long)i * S);
            const int Li = L[i];
            if (Li < 1 || Li > Lmax) continue;
            const int32_t* x = trans_q + (size_t)i * S * S;
            if (x[k * S + d] > x[k * S + s] || x[d * S + k] > x[s * S + k]) dom = 0;
        }
        if (!dom) s_dom = 0;             // benign race: every writer writes 0
        if (!strict) s_strict = 0;
        __syncthreads();
        if (s_dom && (d < s || s_strict)) kept = 0;
    }
    if (threadIdx.x == 0) keep[s] = kept;
}

// map[k] = original index of the k-th kept strategy (ascending), -1 beyond; S_kept = their number.
__global__ void prune_map_kernel(int S, const int32_t* __restrict__ keep, int32_t* __restrict__ map, int32_t* __restrict__ S_kept)
{
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        int n = 0;
        for (int s = 0; s < S; ++s)
            if (keep[s]) map[n++] = s;
        *S_kept = n;
        for (; n < S; ++n) map[n] = -1;
    }
}

__global__ void compact_kernel(int B, int Lmax, int S, int S2, const int32_t* __restrict__ map,
                               const int32_t* __restrict__ time_q, const int32_t* __restrict__ mem_q,
                               const int32_t* __restrict__ trans_q, int32_t* __restrict__ time_o,
                               int32_t* __restrict__ mem_o, int32_t* __restrict__ trans_o)
{
    const long long n1 = (long long)B * Lmax * S2, n2 = (long long)B * S2 * S2;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n1 + n2; e += (long long)gridDim.x * blockDim.x) {
        if (e < n1) {
            const int c = (int)(e % S2);
            const long long il = e / S2;
            time_o[e] = time_q[il * S + map[c]];
            mem_o[e] = mem_q[il * S + map[c]];
        } else {
            const long long f = e - n1;
            const int c = (int)(f % S2), r = (int)((f / S2) % S2);
            const long long i = f / ((long long)S2 * S2);
            trans_o[f] = trans_q[(i * S + map[r]) * S + map[c]];
        }
    }
}

__global__ void expand_kernel(long long n, const int32_t* __restrict__ map, int32_t* __restrict__ plan)
{
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
        const int p = plan[e];
        if (p >= 0) plan[e] = map[p];
    }
}

int blocks_for(long long n) { long long b = (n + 255) / 256; return (int)(b < 1 ? 1 : (b > 148 * 8 ? 148 * 8 : b)); }

}  // namespace

extern "C" {

int galv_prune_strategies(galv_ctx* ctx, const galv_shape* sh, const int32_t* L, const int32_t* time_q,
                          const int32_t* mem_q, const int32_t* trans_q, int32_t* keep, int32_t* map, int32_t* S_kept,
                          void* stream)
{
    if (!ctx) return GALV_ERR_INVALID_ARG;
    if (!sh || sh->B < 1 || sh->S < 1 || sh->S > 256 || sh->Lmax < 1 || !L || !time_q || !mem_q || !trans_q || !keep || !map || !S_kept)
        return galv_set_error(ctx, GALV_ERR_INVALID_ARG, "galv_prune_strategies: bad shape or NULL pointer");
    if (sh->flags & GALV_TRANS_PER_LAYER)
        return galv_set_error(ctx, GALV_ERR_INVALID_ARG, "galv_prune_strategies: one transition matrix per instance only (no GALV_TRANS_PER_LAYER)");
    cudaStream_t st = (cudaStream_t)stream;
    prune_kernel<<<sh->S, 256, 0, st>>>(sh->B, sh->Lmax, sh->S, L, time_q, mem_q, trans_q, keep);
    prune_map_kernel<<<1, 32, 0, st>>>(sh->S, keep, map, S_kept);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? GALV_OK : galv_set_error(ctx, GALV_ERR_CUDA, cudaGetErrorString(e));
}

int galv_compact_tables(galv_ctx* ctx, const galv_shape* sh, int32_t S_kept, const int32_t* map, const int32_t* time_q,
                        const int32_t* mem_q, const int32_t* trans_q, int32_t* time_out, int32_t* mem_out,
                        int32_t* trans_out, void* stream)
{
    if (!ctx) return GALV_ERR_INVALID_ARG;
    if (!sh || sh->B < 1 || sh->S < 1 || sh->Lmax < 1 || S_kept < 1 || S_kept > sh->S || !map || !time_q || !mem_q || !trans_q ||
        !time_out || !mem_out || !trans_out || (sh->flags & GALV_TRANS_PER_LAYER))
        return galv_set_error(ctx, GALV_ERR_INVALID_ARG, "galv_compact_tables: bad shape, S_kept outside 1..S, per-layer trans, or NULL pointer");
    const long long n = (long long)sh->B * sh->Lmax * S_kept + (long long)sh->B * S_kept * S_kept;
    compact_kernel<<<blocks_for(n), 256, 0, (cudaStream_t)stream>>>(sh->B, sh->Lmax, sh->S, S_kept, map, time_q, mem_q, trans_q,
                                                                   time_out, mem_out, trans_out);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? GALV_OK : galv_set_error(ctx, GALV_ERR_CUDA, cudaGetErrorString(e));
}

int galv_expand_plan(galv_ctx* ctx, int32_t B, int32_t Lmax, const int32_t* map, int32_t* plan, void* stream)
{
    if (!ctx) return GALV_ERR_INVALID_ARG;
    if (B < 1 || Lmax < 1 || !map || !plan) return galv_set_error(ctx, GALV_ERR_INVALID_ARG, "galv_expand_plan: bad size or NULL pointer");
    const long long n = (long long)B * Lmax;
    expand_kernel<<<blocks_for(n), 256, 0, (cudaStream_t)stream>>>(n, map, plan);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? GALV_OK : galv_set_error(ctx, GALV_ERR_CUDA, cudaGetErrorString(e));
}

}  // extern "C"
