// What the two opt-in skipping flags of the search would leave out, estimated from the inputs alone.
//
// (The paper has no counterpart: the flags are this library's.)  GALV_SKIP_INFEASIBLE leaves out the tiles of a
// layer that lie wholly below the previous layer's feasibility frontier (no cell of layer l is finite below the
// sum of the layers' smallest mem); that share is exact.  GALV_SKIP_DOMINATED leaves out previous-layer rows that
// lie more than the largest transition entry above the best row in every column of a tile; how many depends on
// the tables the search builds, so the estimate looks at the one layer known beforehand, layer 0, whose rows are
// constants: row s' is counted when time(0,s') exceeds the smallest time(0,.) by more than the largest transition
// entry (or never fits).  One warp per instance.

#include "galv_internal.h"

namespace {

__global__ void estimate_kernel(int B, int Lmax, int S, int M, int tmb, int ntiles_m, long long trans_inst, long long trans_layer,
                                const int32_t* __restrict__ L, const int32_t* __restrict__ time_q, const int32_t* __restrict__ mem_q,
                                const int32_t* __restrict__ trans_q, unsigned long long* __restrict__ counts)
{
    const int lane = threadIdx.x & 31;
    const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (i >= B) return;
    const int Li = L[i];
    if (Li < 1 || Li > Lmax) return;
    const int32_t* tq = time_q + (size_t)i * Lmax * S;
    const int32_t* mq = mem_q + (size_t)i * Lmax * S;
    // tiles below the frontier: layer l (1 .. Li-1) reads layer l-1, whose frontier is the sum of the smallest mem of layers 0 .. l-1
    long long run = 0, below = 0;
    for (int l = 0; l + 1 < Li; ++l) {
        int mn = 0x7fffffff;
        for (int s = lane; s < S; s += 32) mn = min(mn, mq[l * S + s]);
        mn = __reduce_min_sync(0xffffffffu, mn);
        run += mn < 0 ? 0 : mn;
        const long long front = run < (long long)M + 1 ? run : (long long)M + 1;
        const long long n = front / tmb;                       // tiles t with (t+1)*tmb - 1 < front
        below += n < ntiles_m ? n : ntiles_m;
    }
    // rows of layer 0 that cannot win in layer 1
    const int32_t* T = trans_q + (size_t)i * trans_inst + (size_t)trans_layer;      // per-layer matrices: the one paid between layers 0 and 1
    int tmax = 0;
    for (int e = lane; e < S * S; e += 32) tmax = max(tmax, T[e]);
    tmax = __reduce_max_sync(0xffffffffu, tmax);
    int best = 0x7fffffff;
    for (int s = lane; s < S; s += 32)
        if (mq[s] <= M) best = min(best, tq[s]);
    best = __reduce_min_sync(0xffffffffu, best);
    int dom = 0;
    for (int s = lane; s < S; s += 32)
        dom += (mq[s] > M) || ((long long)tq[s] > (long long)best + tmax);
    dom = __reduce_add_sync(0xffffffffu, dom);
    if (lane == 0) {
        atomicAdd(&counts[0], (unsigned long long)below);
        atomicAdd(&counts[1], (unsigned long long)(Li - 1) * ntiles_m);
        atomicAdd(&counts[2], (unsigned long long)dom);
        atomicAdd(&counts[3], (unsigned long long)S);
    }
}

}  // namespace

extern "C" int galv_skip_estimate(galv_ctx* ctx, const galv_shape* sh, const int32_t* L, const int32_t* time_q, const int32_t* mem_q,
                                  const int32_t* trans_q, int64_t* counts, void* stream)
{
    if (!ctx) return GALV_ERR_INVALID_ARG;
    if (!sh || sh->B < 1 || sh->S < 1 || sh->S > 256 || sh->Lmax < 1 || sh->M < 0 || !L || !time_q || !mem_q || !trans_q || !counts)
        return galv_set_error(ctx, GALV_ERR_INVALID_ARG, "galv_skip_estimate: bad shape or NULL pointer");
    DpPlan pl;
    if (!galv_dp_make_plan(ctx, sh, &pl)) return galv_set_error(ctx, GALV_ERR_INVALID_ARG, "galv_skip_estimate: no tiling for this shape");
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = cudaMemsetAsync(counts, 0, 4 * sizeof(int64_t), st);
    if (e == cudaSuccess) {
        estimate_kernel<<<(sh->B + 3) / 4, 128, 0, st>>>(sh->B, sh->Lmax, sh->S, sh->M, pl.tmb, pl.ntiles_m, galv_trans_inst(sh), galv_trans_layer(sh),
                                                         L, time_q, mem_q, trans_q, reinterpret_cast<unsigned long long*>(counts));
        e = cudaGetLastError();
    }
    return e == cudaSuccess ? GALV_OK : galv_set_error(ctx, GALV_ERR_CUDA, cudaGetErrorString(e));
}
