// Optimum extraction and plan backtrack: one warp per search instance.
//
// (Section 3 of the paper: the selector's result is a per-layer parallelism plan.)
// opt = min_s C_last[s][budget] with the lowest s on ties, found by a warp
// shuffle min over packed (cost << 32 | index) keys.  The walk then goes from
// the last layer to the first; the predecessor is read from the argmin table
// when there is one, otherwise it is the lowest s' whose candidate
// C[l-1][m'][s'] + trans(s',s) equals the cell's value minus time(l,s).

#include "galv_internal.h"

namespace {

constexpr int kInf = GALV_INF;

__device__ __forceinline__ unsigned long long warp_min_u64(unsigned long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long w = __shfl_xor_sync(0xffffffffu, v, o);
        v = w < v ? w : v;
    }
    return v;
}

// NJ: strategies per lane (S <= 32 * NJ): the walk's chain of selects, loads and ballots is as long as it has to be.
template <int NJ>
__global__ void backtrack_kernel(int B, int Lmax, int S, int M, int m_pitch, long long trans_inst, long long trans_layer,
                                 const int32_t* __restrict__ L, const int32_t* __restrict__ time_q,
                                 const int32_t* __restrict__ mem_q, const int32_t* __restrict__ trans_q,
                                 const int32_t* __restrict__ C, const uint8_t* __restrict__ A,
                                 const int32_t* __restrict__ C_last, const int32_t* __restrict__ budget,
                                 int32_t* __restrict__ opt_cost, int32_t* __restrict__ plan,
                                 int32_t* __restrict__ mem_used, int32_t* __restrict__ status)
{
    const int lane = threadIdx.x & 31;
    const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (i >= B) return;
    const int st0 = status[i] & ~GALV_STATUS_INFEASIBLE;
    int32_t* pl = plan ? plan + (size_t)i * Lmax : nullptr;
    if (pl)
        for (int l = lane; l < Lmax; l += 32) pl[l] = -1;
    __syncwarp();          // lane 0 overwrites entries other lanes have just cleared
    const int bud = budget ? budget[i] : M;
    // a search whose bounded waits ran out left void tables: not walked either
    const bool skip = (st0 & (GALV_STATUS_BAD_INPUT | GALV_STATUS_OVERFLOW_RISK | GALV_STATUS_TIMEOUT)) != 0 || bud < 0 || bud > M;
    if (skip) {
        if (lane == 0) {
            opt_cost[i] = kInf;
            if (mem_used) mem_used[i] = 0;
            status[i] = st0 | ((bud < 0 || bud > M) ? GALV_STATUS_BAD_INPUT : 0);
        }
        return;
    }
    const int Li = L[i];
    const size_t slice = (size_t)S * m_pitch;

    // optimum at the budget: lowest s among the minima
    unsigned long long key = ~0ull;
    for (int s = lane; s < S; s += 32) {
        const unsigned long long k = ((unsigned long long)(unsigned)C_last[(size_t)i * slice + (size_t)s * m_pitch + bud] << 32) | (unsigned)s;
        key = k < key ? k : key;
    }
    key = warp_min_u64(key);
    const int opt = (int)(key >> 32);
    int s = (int)(key & 0xffffffffu);
    if (opt >= kInf) {
        if (lane == 0) {
            opt_cost[i] = kInf;
            if (mem_used) mem_used[i] = 0;
            status[i] = st0 | GALV_STATUS_INFEASIBLE;
        }
        return;
    }
    if (lane == 0) { opt_cost[i] = opt; status[i] = st0; }
    if (!pl) return;

    const int32_t* tq = time_q + (size_t)i * Lmax * S;
    const int32_t* mq = mem_q + (size_t)i * Lmax * S;
    const int32_t* T0 = trans_q + (size_t)i * trans_inst;
    int m = bud;
    long long used = 0;
    // One dependent memory round trip per layer: the cell's value is carried along (it is the chosen
    // candidate of the step before), and the mem / time rows of the next layer down are fetched, whole,
    // while this layer's candidates are in flight; lane k%32 keeps entries k, k+32, ... (S <= 256).
    int cur = opt;                                             // C[l][m][s] of the cell the walk stands on
    int mrow[NJ], trow[NJ];
#pragma unroll
    for (int j = 0; j < NJ; ++j) {
        const int k = lane + 32 * j;
        mrow[j] = k < S ? mq[(Li - 1) * S + k] : 0;
        trow[j] = k < S ? tq[(Li - 1) * S + k] : 0;
    }
    for (int l = Li - 1; l >= 0; --l) {
        if (lane == 0) pl[l] = s;
        int msel = mrow[0], tsel = trow[0];
#pragma unroll
        for (int j = 1; j < NJ; ++j) {
            msel = (s >> 5) == j ? mrow[j] : msel;
            tsel = (s >> 5) == j ? trow[j] : tsel;
        }
        const int mm = __shfl_sync(0xffffffffu, msel, s & 31);
        const int tt = __shfl_sync(0xffffffffu, tsel, s & 31);
        used += mm;
        if (mm > m) {                  // cannot happen on consistent tables: the cell would be +inf; never index below column 0
            if (lane == 0) status[i] = st0 | GALV_STATUS_BAD_INPUT;
            break;
        }
        if (l == 0) break;
#pragma unroll
        for (int j = 0; j < NJ; ++j) {                          // rows of layer l-1, needed one step from now
            const int k = lane + 32 * j;
            mrow[j] = k < S ? mq[(l - 1) * S + k] : 0;
            trow[j] = k < S ? tq[(l - 1) * S + k] : 0;
        }
        int sp;
        if (A) {
            sp = A[((size_t)i * Lmax + l) * slice + (size_t)s * m_pitch + m];
        } else {
            const int target = cur - tt;
            const int32_t* prev = C + ((size_t)i * Lmax + (l - 1)) * slice + (m - mm);
            const int32_t* T = T0 + (size_t)l * trans_layer;       // paid between layers l-1 and l
            sp = 255;
            // every row's candidate is asked for before the first is looked at: one round trip to memory, not one per 32 rows
            int cv[NJ], tv[NJ];
#pragma unroll
            for (int j = 0; j < NJ; ++j) {
                const int k = lane + 32 * j;
                cv[j] = k < S ? prev[(size_t)k * m_pitch] : kInf;
                tv[j] = k < S ? T[k * S + s] : 0;
            }
#pragma unroll
            for (int j = 0; j < NJ; ++j) {
                if (32 * j >= S) break;
                const bool hit = (cv[j] < kInf) && (cv[j] + tv[j] == target);
                const unsigned b = __ballot_sync(0xffffffffu, hit);
                if (b) {
                    const int src = __ffs(b) - 1;
                    sp = 32 * j + src;
                    cur = __shfl_sync(0xffffffffu, cv[j], src);
                    break;
                }
            }
        }
        if (sp >= S) {                 // cannot happen on consistent tables; stop instead of walking off
            if (lane == 0) status[i] = st0 | GALV_STATUS_BAD_INPUT;
            break;
        }
        m -= mm;
        s = sp;
    }
    if (lane == 0 && mem_used) mem_used[i] = (int32_t)used;
}

}  // namespace

cudaError_t galv_backtrack_launch(const galv_shape* sh, const int32_t* L, const int32_t* time_q,
                                  const int32_t* mem_q, const int32_t* trans_q, const int32_t* C,
                                  const uint8_t* A, const int32_t* C_last, const int32_t* budget,
                                  int32_t* opt_cost, int32_t* plan, int32_t* mem_used, int32_t* status,
                                  cudaStream_t st)
{
    const int warps = 4;
    const dim3 grid((sh->B + warps - 1) / warps), block(warps * 32);
#define GALV_WALK(NJ) backtrack_kernel<NJ><<<grid, block, 0, st>>>( \
        sh->B, sh->Lmax, sh->S, sh->M, sh->m_pitch, galv_trans_inst(sh), galv_trans_layer(sh), L, time_q, mem_q, trans_q, C, A, C_last, budget, \
        opt_cost, plan, mem_used, status)
    if (sh->S <= 32) GALV_WALK(1);
    else if (sh->S <= 64) GALV_WALK(2);
    else if (sh->S <= 128) GALV_WALK(4);
    else GALV_WALK(8);
#undef GALV_WALK
    return cudaGetLastError();
}
