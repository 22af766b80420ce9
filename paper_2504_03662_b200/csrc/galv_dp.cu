// Layer-wise min-plus recurrence of the strategy search on sm_100a.
//
//   C[l][m][s] = time(l,s) + min_{s'} ( C[l-1][m-mem(l,s)][s'] + trans(s',s) )
//
// (Section 3 of the paper: dynamic-programming search over a performance model.)
//
// Per layer the work is a min-plus product G[s][m'] = min_{s'} (Cprev[s'][m'] + T[s'][s])
// that does not depend on mem; mem only shifts where column m' is stored:
// C[l][s][m'+mem(l,s)] = time(l,s) + G[s][m'].  So the kernel tiles like a
// CUDA-core GEMM: an item is (instance, tile of m', block of s); warps own a
// register tile of (TM x 32 columns) x (8 strategies); the previous layer's rows
// and the matching rows of the S x S transition matrix are staged in shared memory
// by tensor-map TMA loads issued by a producer warp, in a multi-stage mbarrier
// pipeline over chunks of s'; the outputs leave through a staging tile and TMA
// bulk stores issued by a store warp.  One fused add-min instruction per
// relaxation; no tensor cores (min-plus is not a multiply-add contraction).
//
// A layer needs the previous one.  With the full table kept, all layers run in one
// cooperative launch: CTAs publish finished tiles in global counters and start a
// tile of the next layer as soon as the tiles it reads are published (bounded
// waits); on the two-layer rolling buffer a tile also waits for the readers of the
// cells it overwrites.  The argmin table is written in such a launch too where its loop
// can work on keys (see the keys-only instantiation); otherwise one launch per layer.
// Either way plain stream work, capturable in a CUDA graph.

#include <cuda.h>

#include <cstring>
#include <type_traits>
#include <cstdlib>

#include "galv_internal.h"

namespace {

constexpr int kInf = GALV_INF;
constexpr int TS = 8;                 // strategies per warp register tile
// Every device-side wait gives up after about a second of waiting (SM clock cycles; checked every 256
// polls): the role sets the error flag and returns, the host sees GALV_STATUS_TIMEOUT, the context stays
// usable.  Time is summed poll interval by poll interval with each interval capped, so that a gap in which
// the whole grid was off the GPU (preemption, time slicing) counts as one interval, not as a timeout.
constexpr long long kWaitLimitCycles = 2000000000LL;
constexpr long long kWaitStepCap = 50000000LL;

struct WaitClock {
    long long last, waited;
    int polls;
    __device__ WaitClock() : last(0), waited(0), polls(0) {}
    // true when the limit ran out
    __device__ bool expired() {
        if ((++polls & 255) != 0) return false;
        const long long now = clock64();
        if (last != 0) {
            const long long step = now - last;
            waited += step < kWaitStepCap ? step : kWaitStepCap;
        }
        last = now;
        return waited > kWaitLimitCycles;
    }
};

// ---------------------------------------------------------------- PTX helpers

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// 2-D tiled TMA load: the box at element coordinates (x, y) of the tensor behind `map` lands densely
// (row-major, box rows of box-width elements) at dst; the box's full byte count is signalled on bar,
// out-of-range elements are filled with zeros.  x * 4 bytes must be a multiple of 16.
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
// 1-D bulk async store shared -> global (both 16-byte aligned, bytes a multiple of 16), tracked in bulk groups.
__device__ __forceinline__ void bulk_s2g(void* dst, const void* src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(smem_u32(src)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ int ld_acquire_gpu(const int32_t* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_relaxed_gpu_add(int32_t* p, int v) {
    asm volatile("red.relaxed.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void red_release_cta_add(int* p, int v) {
    asm volatile("red.release.cta.shared::cta.add.s32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
}
__device__ __forceinline__ void st_release_cta(int* p, int v) {
    asm volatile("st.release.cta.shared::cta.s32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
}
__device__ __forceinline__ int ld_acquire_cta(const int* p) {
    int v;
    asm volatile("ld.acquire.cta.shared::cta.s32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)) : "memory");
    return v;
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false when the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    WaitClock wc;
    while (!mbar_try_wait(bar, parity))
        if (wc.expired()) return false;
    return true;
}
// The same for the role warps, which wait long and often: a warp that spins on try_wait takes issue
// slots and ALU cycles from the four consumer warps on its scheduler, so it sleeps between polls.
__device__ __forceinline__ bool mbar_wait_idle(uint64_t* bar, uint32_t parity) {
    WaitClock wc;
    while (!mbar_try_wait(bar, parity)) {
        if (wc.expired()) return false;
        __nanosleep(100);
    }
    return true;
}
// 1-D bulk async copy global -> shared, completion counted in bytes on an mbarrier.
// dst, src 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// ---------------------------------------------------------------- validation / schedule

// One CTA per instance: entries >= 0, L in range, worst-case path sum below kInf.
// tl: entries between the transition matrices of consecutive layers (0: one matrix per instance; S*S: matrix l
// is paid between layers l-1 and l, matrix 0 unused).
__global__ void validate_kernel(int B, int Lmax, int S, int M, long long tl, const int32_t* __restrict__ L,
                                const int32_t* __restrict__ time_q, const int32_t* __restrict__ mem_q,
                                const int32_t* __restrict__ trans_q, int32_t* __restrict__ status,
                                int32_t* __restrict__ maxmem, int32_t* __restrict__ minmem_l, int32_t* __restrict__ front)
{
    const int i = blockIdx.x;
    __shared__ long long s_sum;
    __shared__ int s_tmax, s_bad, s_mmax;
    if (threadIdx.x == 0) { s_sum = 0; s_tmax = 0; s_bad = 0; s_mmax = 0; }
    __syncthreads();
    const int Li = L[i];
    if (Li < 1 || Li > Lmax) {
        if (threadIdx.x == 0) status[i] = GALV_STATUS_BAD_INPUT;
        return;
    }
    long long sum = 0;
    int bad = 0, tmax = 0, mmax = 0;
    const int32_t* t = time_q + (size_t)i * Lmax * S;
    const int32_t* mq = mem_q + (size_t)i * Lmax * S;
    for (int l = threadIdx.x; l < Li; l += blockDim.x) {
        int mx = 0;
        for (int s = 0; s < S; ++s) {
            const int tv = t[l * S + s], mv = mq[l * S + s];
            bad |= (tv < 0) | (mv < 0);
            mx = max(mx, tv);
            mmax = max(mmax, mv);
        }
        sum += mx;
    }
    const int32_t* x = trans_q + (size_t)i * (tl ? (size_t)Lmax * S * S : (size_t)S * S);
    const int xl0 = tl ? 1 : 0, xl1 = tl ? Li : 1;            // matrices in use
    for (long long k = threadIdx.x; k < (long long)(xl1 - xl0) * S * S; k += blockDim.x) {
        const int v = x[(size_t)xl0 * S * S + k];
        bad |= (v < 0);
        tmax = max(tmax, v);
    }
    atomicAdd(reinterpret_cast<unsigned long long*>(&s_sum), static_cast<unsigned long long>(sum));
    atomicMax(&s_tmax, tmax);
    atomicMax(&s_mmax, mmax);
    if (bad) atomicOr(&s_bad, 1);
    __syncthreads();
    if (threadIdx.x == 0) {
        int st = 0;
        if (s_bad) st = GALV_STATUS_BAD_INPUT;
        else if (s_sum + (long long)(Li - 1) * s_tmax >= (long long)kInf) st = GALV_STATUS_OVERFLOW_RISK;
        status[i] = st;
        // largest shift of a stored row over the valid instances (M+1 stands for "fills the whole row")
        if (st == 0) {
            atomicMax(maxmem, min(s_mmax, M + 1));
            atomicMax(maxmem + 1, s_tmax);                     // largest transition entry: decides the 16-bit path
        }
        s_bad = st;
    }
    __syncthreads();
    if (s_bad == 0) {
        for (int l = threadIdx.x; l < Li; l += blockDim.x) {      // smallest mem of each layer over the valid instances
            int mn = 0x7fffffff;
            for (int s = 0; s < S; ++s) mn = min(mn, mq[l * S + s]);
            atomicMin(&minmem_l[l], mn);
            if (front) front[(size_t)i * Lmax + l] = mn;
        }
        if (front) {
            // feasibility frontier: no cell of layer l is finite below the sum of the layers' smallest mem
            __syncthreads();
            if (threadIdx.x == 0) {
                long long run = 0;
                for (int l = 0; l < Li; ++l) {
                    run += front[(size_t)i * Lmax + l];
                    front[(size_t)i * Lmax + l] = (int32_t)min(run, (long long)M + 1);
                }
            }
        }
    }
}

// Inclusive prefix sum of one value per thread over a block of 1024 threads; *total = the block's sum.
__device__ long long block_scan_1024(long long v, long long* warp_sums, long long* total)
{
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const long long t = __shfl_up_sync(0xffffffffu, v, off);
        if (lane >= off) v += t;
    }
    if (lane == 31) warp_sums[wid] = v;
    __syncthreads();
    if (wid == 0) {
        long long w = warp_sums[lane];
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const long long t = __shfl_up_sync(0xffffffffu, w, off);
            if (lane >= off) w += t;
        }
        warp_sums[lane] = w;
    }
    __syncthreads();
    if (wid > 0) v += warp_sums[wid - 1];
    *total = warp_sums[31];
    __syncthreads();
    return v;
}

// Single CTA of 1024 threads: nactive[l] = valid instances with L > l; order = valid instances, longest first.
// scratch = hist[Lmax+2] | fill[Lmax+2], zeroed by the host before the launch.
// ntiles[l] = tiles of tmb columns per instance that can store anything in layer l: column m' lands at
// m' + mem(l,s) <= M, so tiles starting above M - (smallest mem of the layer) are left out (at least one
// tile stays: it also writes the cells no column maps to).
// istart[l] = work items (instance, tile, s-block) of layers 1 .. l-1: the items of all layers in one sequence.
// tcount[l][t] = layers 1 .. l whose items include tile t.
__global__ void __launch_bounds__(1024) schedule_kernel(int B, int Lmax, int M, int tmb, int ntiles_m, int nsb, const int32_t* __restrict__ L,
                                const int32_t* __restrict__ status, int32_t* __restrict__ order, int32_t* __restrict__ nactive,
                                int32_t* __restrict__ scratch, const int32_t* __restrict__ minmem_l, int32_t* __restrict__ ntiles,
                                long long* __restrict__ istart, int32_t* __restrict__ tcount, int p16_possible,
                                int32_t* __restrict__ maxmem)
{
    __shared__ long long warp_sums[32];
    // The packed 16-bit path needs every trans entry, and twice the largest plus one, to fit 16 bits.
    if (threadIdx.x == 0) maxmem[2] = (p16_possible && maxmem[1] <= 32767) ? 1 : 0;
    int32_t* hist = scratch;
    int32_t* fill = scratch + Lmax + 2;
    for (int i = threadIdx.x; i < B; i += blockDim.x)
        if (status[i] == 0) atomicAdd(&hist[L[i]], 1);
    for (int l = threadIdx.x; l <= Lmax; l += blockDim.x) {
        int nt = 1;
        if (l < Lmax && minmem_l[l] <= M) nt = min(ntiles_m, (M - minmem_l[l]) / tmb + 1);
        ntiles[l] = max(1, nt);
    }
    __syncthreads();
    {
        long long carry = 0, total;                    // instances with L > l: a sum from the top layer down
        for (int base = 0; base <= Lmax; base += 1024) {
            const int l = Lmax - (base + (int)threadIdx.x);
            const long long h = l >= 0 ? hist[l] : 0;
            const long long incl = block_scan_1024(h, warp_sums, &total);
            if (l >= 0) nactive[l] = (int32_t)(carry + incl - h);
            carry += total;
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < B; i += blockDim.x)
        if (status[i] == 0) {
            const int Li = L[i];
            order[nactive[Li] + atomicAdd(&fill[Li], 1)] = i;   // instances longer than Li come first
        }
    for (int t = threadIdx.x; t < ntiles_m; t += blockDim.x) {
        int run = 0;
        tcount[t] = 0;
        for (int l = 1; l < Lmax; ++l) {
            run += t < ntiles[l];
            tcount[(size_t)l * ntiles_m + t] = run;
        }
    }
    {
        long long carry = 0, total;
        if (threadIdx.x == 0) istart[0] = 0;
        for (int base = 1; base <= Lmax; base += 1024) {
            const int l = base + (int)threadIdx.x;
            const long long v = l < Lmax ? (long long)nactive[l] * ntiles[l] * nsb : 0;
            const long long incl = block_scan_1024(v, warp_sums, &total);
            if (l <= Lmax) istart[l] = carry + incl - v;
            carry += total;
        }
    }
}

// ---------------------------------------------------------------- base layer

// C[0][s][m] = time(0,s) if mem(0,s) <= m else INF; pad columns INF; A = 255.
__global__ void base_layer_kernel(DpArgs a)
{
    const int i = blockIdx.z, s = blockIdx.y;
    if (a.status[i] != 0) return;
    const int tt = a.time_q[(size_t)i * a.Lmax * a.S + s];
    const int mm = a.mem_q[(size_t)i * a.Lmax * a.S + s];
    const size_t row = ((size_t)i * a.S + s) * a.m_pitch;
    int32_t* out = a.C ? a.C + ((size_t)i * a.Lmax * a.S + s) * a.m_pitch : a.roll + row;
    uint8_t* ao = a.A ? a.A + ((size_t)i * a.Lmax * a.S + s) * a.m_pitch : nullptr;
    for (int m = blockIdx.x * blockDim.x + threadIdx.x; m < a.m_pitch; m += gridDim.x * blockDim.x) {
        const int v = (m <= a.M && mm <= m) ? tt : kInf;
        out[m] = v;
        if (ao) ao[m] = 255;
    }
}

// ---------------------------------------------------------------- reference layer kernel (one thread per cell)

__global__ void layer_reference_kernel(DpArgs a, int l)
{
    const int mchunks = (a.m_pitch + blockDim.x - 1) / blockDim.x;
    const int oi = blockIdx.x / mchunks;
    if (oi >= a.nactive[l]) return;
    const int i = a.order[oi], s = blockIdx.y;
    const int m = (blockIdx.x % mchunks) * blockDim.x + threadIdx.x;
    if (m >= a.m_pitch) return;
    const size_t slice = (size_t)a.S * a.m_pitch;
    const int32_t* prev = a.C ? a.C + ((size_t)i * a.Lmax + (l - 1)) * slice : a.roll + ((size_t)((l - 1) & 1) * a.B + i) * slice;
    int32_t* out = a.C ? a.C + ((size_t)i * a.Lmax + l) * slice : a.roll + ((size_t)(l & 1) * a.B + i) * slice;
    const int32_t* T = a.trans_q + (size_t)i * a.trans_inst + (size_t)l * a.trans_layer;
    const int mm = a.mem_q[((size_t)i * a.Lmax + l) * a.S + s];
    const int tt = a.time_q[((size_t)i * a.Lmax + l) * a.S + s];
    int best = kInf, arg = 255;
    if (m <= a.M && mm <= m) {
        const int mp = m - mm;
        for (int sp = 0; sp < a.S; ++sp) {
            const int c = prev[(size_t)sp * a.m_pitch + mp];
            if (c < kInf) {
                const int v = c + T[sp * a.S + s];
                if (v < best) { best = v; arg = sp; }
            }
        }
    }
    const int v = best < kInf ? best + tt : kInf;
    out[(size_t)s * a.m_pitch + m] = v;
    if (a.A) a.A[(((size_t)i * a.Lmax + l) * a.S + s) * a.m_pitch + m] = (uint8_t)arg;
}

// ---------------------------------------------------------------- packed trans rows (16-bit path)

// trans_p[i][(l)][p][s] = T[a][s] | T[a + 2][s] << 16 with a = 4 * (p / 2) + p % 2: packed row p pairs rows a and a + 2,
// as the rebase does (one lane of a column takes the even rows, one the odd).  The low 16 bits of each entry; used only
// when they all fit.
__global__ void pack_trans_kernel(long long n_mats, int S, const int32_t* __restrict__ trans_q, uint32_t* __restrict__ trans_p)
{
    const long long n = n_mats * (S / 2) * S;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
        const int s = (int)(e % S);
        const long long mq = e / S;
        const int q = (int)(mq % (S / 2));
        const long long mat = mq / (S / 2);
        const int32_t* T = trans_q + mat * S * S;
        const int ra = 4 * (q >> 1) + (q & 1);
        trans_p[e] = ((uint32_t)T[ra * S + s] & 0xffffu) | ((uint32_t)T[(ra + 2) * S + s] << 16);
    }
}

// trans_k = trans_q with every entry << 6 when keys are possible (largest entry of the valid instances < 2^24, so that
// rebased cost + entry, shifted, stays below 2^31), else a plain copy; maxmem[3] tells the layer kernels which.
__global__ void key_trans_kernel(long long n, const int32_t* __restrict__ trans_q, int32_t* __restrict__ trans_k, int32_t* __restrict__ maxmem)
{
    const int sh = maxmem[1] < (1 << 24) ? 6 : 0;
    if (blockIdx.x == 0 && threadIdx.x == 0) maxmem[3] = sh != 0;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
        const int v = trans_q[e];
        trans_k[e] = v < 0 ? v : (int)((unsigned)v << sh);     // negative entries belong to flagged instances: never read
    }
}

// ---------------------------------------------------------------- tiled layer kernel
//
// Work items are (layer, instance, m'-tile, s-block), numbered layer by layer.  CTAs take them one
// at a time from a global counter, so the SMs stay evenly loaded whatever the items weigh, and items
// taken at about the same time mostly share the instance (its trans rows stay in L2).  Warp roles:
//   warp NC (producer): takes the next item and posts its record in a small ring in shared memory
//       for the other roles; then for every chunk (item, k-chunk of s') waits for a free stage and
//       copies KS rows of the previous layer's slice and the matching rows of trans into it (TMA);
//   warp NC+1 (helper): stages each item's record (mem and time row of the s-block, instance)
//       next to the item's last chunk, and writes the cells no column maps to (m < mem(l,s))
//       and the pad columns;
//   warp NC+2 (store warp): sends the finished item's outputs from a staging tile in shared memory
//       to the table, one bulk async store (TMA) per row, while the consumers already work on the
//       next item.  The SM's store port takes 32 bytes per clock whoever feeds it; fed by plain
//       stores of the consumers it also holds up their shared-memory loads, the TMA unit reads
//       shared memory on its own path;
//   warp NC+3 (publisher): with all layers in one launch, makes the finished tiles known to the other
//       SMs (a.tile_done).  That takes fences, and a fence lasts thousands of cycles while the SM's
//       stores are in flight; here they delay nobody and cover several items at once;
//   warps 0..NC-1 (consumers): warp (ms, sg) keeps a TM x 8 register tile per lane
//       (columns m' = tile + ms*32*TM + j*32 + lane, strategies sg*8 .. sg*8+7), waits for the
//       stage, runs one fused add-min per relaxation, releases the stage, and after the last
//       chunk adds time(l,s) and writes its tile into the staging tile, row s shifted by
//       mem(l,s) mod 4 so that column m' + mem(l,s) of the table is 16-byte aligned with it.
// Stages are handed over with mbarriers (full: bytes landed and record written; empty: every consumer
// warp done; out_full for the staging tile, a counter for its drain), so there is no block-wide barrier in the
// loop.  Every wait is bounded; a wait that runs out sets the error flag and the role returns.

constexpr int kMaxStages = 4;
constexpr int kStaticSmemReserve = 512;                // the kernel's static shared memory (barriers, item ring, counters), rounded up

struct ItemPos { int oi, mt, sb; };

// nt = tiles per instance in the layer at hand (the trailing tiles that cannot store anything are left out)
__device__ __forceinline__ ItemPos item_at(long long item, int nt, int nsb) {
    const int per = nt * nsb;
    ItemPos p;
    p.oi = (int)(item / per);
    const int r = (int)(item - (long long)p.oi * per);
    p.mt = r / nsb;
    p.sb = r - p.mt * nsb;
    return p;
}

// Item records in flight: the producer runs at most (stages + 3) items ahead of the store warp, and
// the store warp at most kPublishLag items ahead of the publisher.
constexpr int kPublishLag = 5;
constexpr int kDescRing = 16;

// Shared memory: NST stages of [KS][TMB] previous-layer values + [KS][SB] trans values, then per
// stage a small record the producer fills for the item whose last chunk sits in that stage:
// mem(l,s) and time(l,s) of the s-block and the instance index; then the staging tile of the
// outputs and its header.
//
// Packed 16-bit variant (P16): min-plus is invariant under a shift of all candidates of a column, and a
// candidate more than the largest trans entry above the column's smallest previous-layer value can never
// win.  So per column m' the previous-layer values are rebased to d = min(c - min_s' c, maxT + 1), which fits
// 16 bits whenever 2 * maxT + 1 does, and two of them (rows 2q and 2q+1) share a register, as do the two
// trans entries T[2q][s], T[2q+1][s] (packed once per call).  One __viaddmin_u16x2 then does two relaxations;
// the result is min(low half, high half) + the column's base.  Exact: only differences are formed, nothing
// is rounded, clamped candidates stay above every possible winner.  The whole tile (all S rows) comes from
// the table as int32 into ONE buffer and is rebased by the consumer warps into one of two packed stages, so
// the next tile's load runs under this tile's inner loop.  Warps NC+4.. are further store warps there.
//
// Dominated rows left out (DOM, opt-in): the same bound says that a previous-layer row clamped in every column
// of a warp group's 128-column tile contributes nothing to that tile.  The packed variant notes the live row
// pairs while it rebases; the 32-bit variant (all S <= 64 rows in one stage) scans its columns first.  Either
// way the group ORs its live rows together, meets at a barrier and relaxes only those.  Same results.
//
// Roles of a CTA and what each hand-over is (every wait is bounded; a wait that runs out sets a.err and the role leaves):
//   producer (warp NC)      takes the next item from the global counter, posts its record in desc[] (desc_count), waits for
//                           the tiles of layer l-1 it reads (tile_done[], acquire at gpu scope; rolling buffer: also for the
//                           readers of the cells it overwrites, then deps_ok), waits for the stage (empty_bar[stage], all
//                           consumer warps) and issues the TMA loads, which complete on full_bar[stage] (1 arrival + bytes).
//   helper (warp NC+1)      reads the record, writes mem / time of the s-block into the stage's item record, gives
//                           full_bar[stage] its second arrival; for a first tile writes the cells no tile stores (fill_count).
//   consumers (0 .. NC-1)   wait full_bar[stage], relax, arrive on empty_bar[stage]; wait until the store warps have read the
//                           previous item out of the staging tile (out_drained), write this item's outputs there, arrive on
//                           out_full.  conv_bar[column group]: hand-overs inside a group (rebase, keys, live rows).
//   store warp (NC+2)       waits out_full, orders the staging writes for the async proxy, issues the bulk stores; once they
//   (+ NC+4.. when packed)  have READ the staging tile: out_drained.  One launch over all layers: once they are COMPLETE, and
//                           the helper's fill and the other store warps' rows (drained_b) as well: drained_count.
//   publisher (NC+3)        one proxy fence and one gpu-scope fence for all items handed over since its last round, then one
//                           relaxed add per item to tile_done[instance][tile]; published_count keeps the store warp within
//                           kPublishLag records of it (the records live in a ring).
//   end                     the producer posts a record with layer -1 and arrives on full_bar; the consumers pass it on through
//                           out_full; the store warp sets store_exit for the publisher.
// The roles are kept in one function body on purpose: split into member functions of a context object the same code ran
// 2.6 % (packed loop) to 30 % (keys loop) slower, so the kernel stays as measured.
template <int TM, int NSG, int NMS, bool ARG, bool MULTI, bool P16 = false, bool DOM = false, bool KEY = false>
__global__ void __launch_bounds__((NSG * NMS + (P16 ? (DOM ? 7 : 5) : 4)) * 32, 1) layer_tiled_kernel(const DpArgs a, const DpPlan pl, const int l_first, const int l_last_arg,
                                                                              const __grid_constant__ CUtensorMap map_c,
                                                                              const __grid_constant__ CUtensorMap map_t)
{
    constexpr int NC = NSG * NMS;                         // consumer warps
    constexpr int SB = NSG * TS;                          // strategies per item
    constexpr int TMB = NMS * 32 * TM;                    // columns per item
    constexpr int BOXC = 32 * TM * ((NMS % 2 == 0 && 64 * TM <= 256) ? 2 : 1);   // columns per TMA box (box extents are <= 256)
    constexpr int NBOX = TMB / BOXC;
    constexpr int META = 2 * SB + 4 + ((DOM && !P16) ? ((2 * NMS + 3) & ~3) : 0);   // 32-bit loop without dominated rows: two words of live rows per
                                                                                    // column group; a multiple of 4 (the record is read 16 bytes at a time)
    static_assert(META % 4 == 0, "item records are read with 16-byte loads");
    constexpr int RS = TMB + 4;                           // staging row: TMB columns + room for the shift
    // Packed path: the raw tile comes in boxes of 128 columns with 16 more on the right, and the packed rows are 16
    // words longer than the tile: row pitches of 16 mod 32 words, so that the two lanes that share a column (one the
    // even rows, one the odd rows) and the two packed rows they write fall into different banks.  (The wider boxes
    // read an eighth more of the table: 1 % slower where dominated rows are left out and the table traffic is the bound.)
    constexpr int CB = 128, PBOX = CB + 16, NRB = TMB / CB, PP = TMB + 16;
    static_assert(!P16 || TMB % CB == 0, "whole raw boxes");
    constexpr bool ARGR = ARG && !KEY;                    // the minimising row is carried in registers of its own (not inside a key)
    constexpr int KU = ARGR ? 4 : 16;                     // k-steps per trip of the inner loop
    constexpr int NSW = P16 ? (DOM ? 4 : 2) : 1;          // store warps: the packed path's items are short enough for one
                                                          // warp's row-by-row issue (about 10k cycles a tile) to hold them up;
                                                          // with dominated rows left out the drain of the staging tile is
                                                          // what the next tile waits for
    constexpr int RPW = 64 / NSW;                         // staging rows (of at most 64) per store warp
    static_assert(TMB % BOXC == 0 && BOXC % (32 * TM) == 0, "a warp's columns must sit inside one box");
    static_assert(!(ARG && P16) && (!P16 || MULTI), "the packed path keeps no argmin and runs all layers in one launch");
    static_assert(!KEY || (ARG && MULTI && !P16 && !DOM), "the keys-only instantiation writes an argmin table, all layers in one launch");

    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kMaxStages];
    __shared__ __align__(8) uint64_t out_full;             // staging tile written (all consumer warps)
    __shared__ int out_drained;                            // items whose staging tile the store warp has read out: a plain
                                                           // counter, its acquire load returns ten times sooner than a barrier wait
    __shared__ int fill_count;                             // helper -> store warp: first tiles whose unreachable cells are written
    __shared__ int4 desc[kDescRing];                       // item records: layer (-1: no more items), instance, tile, s-block
    __shared__ int desc_count;                             // records posted so far
    __shared__ int drained_count, published_count;         // store warp -> publisher: items whose stores are complete; and back
    __shared__ int store_exit;                             // the store warp has left
    __shared__ int deps_ok;                                // rolling buffer: items whose dependency wait the producer has passed
    __shared__ __align__(8) uint64_t conv_bar[16];         // packed path: the warps of a column group have rebased their columns
    __shared__ int drained_b;                              // further store warps -> first: items whose rows they have stored completely (one count each)

    // Which of the two one-launch kernels runs is decided on the device (largest transition entry).
    if (MULTI && !KEY && (a.maxmem[2] != 0) != P16) return;
    // Argmin table: the keys-only kernel (one launch over all layers) runs when the transition entries are small
    // enough for keys; the launches per layer that follow it then have nothing left to do.
    if (KEY && a.maxmem[3] == 0) return;
    if (ARG && !KEY && a.keyed_multi && a.maxmem[3] != 0) return;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int S = a.S, M = a.M, m_pitch = a.m_pitch;
    const int KS = P16 ? S : pl.ks, NKC = P16 ? 1 : pl.nkc, NST = P16 ? 2 : pl.nst;
    // Argmin table with keys (S <= 64, all rows of a tile in one stage, transition entries below 2^24): the previous-layer
    // values of a tile are rebased per column and rewritten as (difference << 6 | row), the transition entries come
    // shifted by 6 bits, and ONE fused add-min per relaxation carries cost and lowest minimising row together.
    const bool keyed = KEY || (ARG && !DOM && !P16 && a.keyed && a.maxmem[3] != 0);
    const int Q = S / 2;                                   // packed path: row pairs
    const int l_last = MULTI ? l_last_arg : l_first + 1;  // single-layer instantiation: loops over l run once
    int32_t* const tile_done = MULTI ? a.tile_done : nullptr;

    // Layers l_first .. l_last-1.  One layer per launch, or all of them in one cooperative launch
    // (a.tile_done set): then an item of layer l starts once the tiles of layer l-1 it reads are
    // complete, which their store warps publish in a.tile_done (see the producer and the store warp).
    // Items are handed out in increasing order and read only items of the layer before, so the
    // lowest unfinished item can always run: the waits end.

    // stage: NBOX boxes of [KS][BOXC] previous-layer values, then [KS][SB] trans values; 128-byte multiples.
    // Packed path: the raw tile (NRB boxes of [S][PBOX]) first, then two stages of [Q][PP] packed values,
    // [Q][SB] packed trans entries, [TMB] column bases and one word per consumer warp (row pairs alive in its columns).
    int32_t* const raw0 = reinterpret_cast<int32_t*>(smem_raw);
    const int raw_elems = P16 ? ((S * PBOX * NRB + 31) & ~31) : 0;
    int32_t* const stage0 = raw0 + raw_elems;
    const int stage_elems = P16 ? ((Q * PP + Q * SB + TMB + NC + 31) & ~31) : ((KS * (TMB + SB) + 31) & ~31);
    int32_t* const meta0 = stage0 + NST * stage_elems;
    // staging tile [SB][RS] + its header: mem(l,s) per row, instance, last-layer flag
    int32_t* const stg0 = meta0 + ((NST * META + 31) & ~31);
    int32_t* const hdr0 = stg0 + SB * RS;

    if (tid == 0) {
        for (int k = 0; k < NST; ++k) { mbar_init(&full_bar[k], 2); mbar_init(&empty_bar[k], NC); }
        mbar_init(&out_full, NC);
        for (int k = 0; k < NMS; ++k) mbar_init(&conv_bar[k], NSG);
        out_drained = 0;
        fill_count = 0;
        desc_count = 0;
        drained_count = 0;
        published_count = 0;
        store_exit = 0;
        deps_ok = 0;
        drained_b = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const size_t slice = (size_t)S * m_pitch;
    // Bounded wait (producer, helper) until the stage of chunk n may be refilled.  Packed path: until every
    // consumer warp has rebased the item before, which frees the raw buffer and, two items back, the stage.
    auto stage_free = [&](int n) -> bool {
        if (P16) return n < 1 || mbar_wait_idle(&empty_bar[0], (n - 1) & 1);
        return n < NST || mbar_wait_idle(&empty_bar[n % NST], ((n / NST) - 1) & 1);
    };

    if (warp == NC) {
        // ------------------------------------------------------------ producer
        const bool tma_t = pl.tma_t != 0;                 // trans rows 16-byte aligned: one box per chunk
        const int inst_rows = a.C ? a.Lmax * S : S;
        // tiles of the previous layer an item reads: its own and, because rows are stored shifted by
        // up to the largest mem, the kdep before it
        const int kdep = tile_done ? (min(*a.maxmem, M) + TMB - 1) / TMB : 0;
        int n = 0;                                        // chunk counter
        // this launch's items are g_base .. g_end-1 of the sequence over all layers
        const long long g_base = a.istart[l_first], g_end = a.istart[l_last];
        unsigned long long* const work = a.work + (MULTI ? 0 : l_first);
        // Global loads and atomics come back after thousands of cycles while the SM's stores are in
        // flight, so the next item is taken and decoded in the shadow of this item's waits.
        int nl = l_first, nt = a.ntiles[l_first], ntp = a.ntiles[l_first - 1];   // decoder state: layer, its tiles, the tiles of the layer before
        long long lbeg = g_base, lend = a.istart[l_first + 1];
        struct Item { int l, i, mt, sb, ntp; };
        auto grab = [&]() -> long long {                  // lane 0 holds the result
            return lane == 0 ? g_base + (long long)atomicAdd(work, 1ull) : 0;
        };
        auto decode = [&](long long g0) -> Item {          // items arrive in increasing order
            const long long g = __shfl_sync(0xffffffffu, g0, 0);
            Item r = {-1, 0, 0, 0, 0};
            if (g < g_end) {
                while (g >= lend) { ++nl; lbeg = lend; lend = a.istart[nl + 1]; ntp = nt; nt = a.ntiles[nl]; }
                const ItemPos p = item_at(g - lbeg, nt, pl.nsb);
                r.l = nl; r.i = a.order[p.oi]; r.mt = p.mt; r.sb = p.sb; r.ntp = ntp;
            }
            return r;
        };
        Item cur = decode(grab());
        for (int it = 0;; ++it) {
            const int l = cur.l, i = cur.i;
            const bool last = l < 0;
            const ItemPos pos = {0, cur.mt, cur.sb};
            if (lane == 0) {
                desc[it % kDescRing] = make_int4(l, i, pos.mt, pos.sb);
                __threadfence_block();
                *reinterpret_cast<volatile int*>(&desc_count) = it + 1;
            }
            __syncwarp();
            if (last) {
                // the consumers learn it through a stage that carries no data
                const int st = n % NST;
                if (!stage_free(n)) {
                    if (lane == 0) atomicExch(a.err, 1);
                    return;
                }
                if (lane == 0) mbar_arrive(&full_bar[st]);
                return;
            }
            const long long g_next = grab();              // lands while the dependencies are polled
            const int row0 = a.C ? (l - 1) * S : ((l - 1) & 1) * a.B * S;      // row of (instance 0, layer l-1, s'=0)
            const int m0 = pos.mt * TMB;
            if (MULTI && tile_done && l > 1) {
                // bounded wait for the tiles of layer l-1 (all their s-blocks) this item reads
                // = s-blocks x the layers up to l-1 that ran the tile (trailing tiles are left out layer by layer)
                const int32_t* const ran = a.tcount + (size_t)(l - 1) * pl.ntiles_m;
                // One lane per tile polls with acquire loads; the warp barrier below orders them before
                // lane 0's TMA loads.  The writes the counters stand for were pushed through the publisher's
                // proxy fence before its release, so no fence is needed here (it would cost this warp
                // thousands of cycles per item while the SM's own stores are in flight).
                // With the two-layer rolling buffer this item overwrites what layer l-2 left there, which the
                // items of layer l-1 on this tile and the kdep after it still read: it waits for those too.
                bool ok = true;
                const int tlast = min(pos.mt + (a.C ? 0 : kdep), cur.ntp - 1);   // tiles the previous layer did not run store nothing
                for (int t0 = max(0, pos.mt - kdep); t0 <= tlast && ok; t0 += 32) {
                    const int t = t0 + lane;
                    if (t <= tlast) {
                        const int32_t* c = tile_done + (size_t)i * pl.ntiles_m + t;
                        WaitClock wc;
                        const int need = ran[t] * pl.nsb;
                        while (ld_acquire_gpu(c) < need) {
                            if (wc.expired()) { ok = false; break; }
                            __nanosleep(100);
                        }
                    }
                    ok = __all_sync(0xffffffffu, ok);
                }
                __syncwarp();
                if (!ok) {
                    if (lane == 0) atomicExch(a.err, 1);
                    return;
                }
            }
            if (MULTI && tile_done && !a.C && lane == 0) st_release_cta(&deps_ok, it + 1);   // the helper may write into the buffer now
            const int sb0 = pos.sb * SB;
            const int sbw = min(SB, S - sb0);             // strategies of this block that exist
            const int yc = row0 + i * inst_rows;
            const int32_t* T = ((ARG && a.keyed) ? a.trans_k : a.trans_q) + (size_t)i * a.trans_inst + (size_t)l * a.trans_layer + sb0;
            const int yt = a.trans_layer ? (i * a.Lmax + l) * S : i * S;     // row of trans(0, .) in the tensor map
            // a tile wholly below the previous layer's feasibility frontier reads nothing but +inf: no loads
            const bool skip = a.front && m0 + TMB - 1 < a.front[(size_t)i * a.Lmax + (l - 1)];
            if constexpr (P16) {
                // one raw tile and one stage of packed trans rows per item; the raw buffer is free once every
                // consumer warp has rebased the item before (which also means the stage of two items ago is free)
                const int st = n & 1;
                if (!stage_free(n)) {
                    if (lane == 0) atomicExch(a.err, 1);
                    return;
                }
                if (skip) {
                    if (lane == 0) mbar_arrive(&full_bar[st]);
                } else if (!((a.withhold & 1) && blockIdx.x == 0 && n == 0) && lane == 0) {
                    mbar_expect_tx(&full_bar[st], (uint32_t)(S * PBOX * NRB + Q * SB) * 4u);
#pragma unroll
                    for (int bx = 0; bx < NRB; ++bx)
                        tma_load_2d(raw0 + bx * S * PBOX, &map_c, m0 + bx * CB, yc, &full_bar[st]);
                    tma_load_2d(stage0 + st * stage_elems + Q * PP, &map_t, 0,
                                (a.trans_layer ? i * a.Lmax + l : i) * Q, &full_bar[st]);
                }
                __syncwarp();
                ++n;
            }
            for (int kc = 0; kc < (P16 ? 0 : NKC); ++kc, ++n) {
                const int st = n % NST;
                if (!stage_free(n)) {
                    if (lane == 0) atomicExch(a.err, 1);
                    return;
                }
                if (skip) {
                    if (lane == 0) mbar_arrive(&full_bar[st]);
                    __syncwarp();
                    continue;
                }
                if (a.withhold && blockIdx.x == 0 && n == 0) continue;   // test hook: a stage that never fills
                const int k0 = kc * KS;
                int32_t* cs = stage0 + st * stage_elems;
                int32_t* ts = cs + KS * TMB;
                if (!tma_t) {
                    // unaligned trans rows: plain copies by this warp, published by the arrive below
                    const int kn = min(KS, S - k0);
                    for (int e = lane; e < kn * sbw; e += 32) {
                        const int r = e / sbw, c = e - r * sbw;
                        ts[r * SB + c] = __ldg(T + (size_t)(k0 + r) * S + c);
                    }
                    __syncwarp();
                }
                if (lane == 0) {
                    // boxes always deliver their full size (zeros beyond the tensor's edge)
                    mbar_expect_tx(&full_bar[st], (uint32_t)KS * (uint32_t)(TMB + (tma_t ? SB : 0)) * 4u);
#pragma unroll
                    for (int bx = 0; bx < NBOX; ++bx)
                        tma_load_2d(cs + bx * KS * BOXC, &map_c, m0 + bx * BOXC, yc + k0, &full_bar[st]);
                    if (tma_t) tma_load_2d(ts, &map_t, sb0, yt + k0, &full_bar[st]);
                }
                __syncwarp();
            }
            // Only now the next item: its decoding waits for loads of its own (layer bounds, instance index),
            // which must not sit between this item's dependency wait and its loads.
            cur = decode(g_next);
        }
    }
    if (warp == NC + 1) {
        // ------------------------------------------------------------ helper
        int n = 0, nfilled = 0;
        for (int it = 0;; ++it) {
            {
                WaitClock wc;                             // the producer posts the item's record
                while (*reinterpret_cast<volatile int*>(&desc_count) <= it) {
                    if (wc.expired()) {
                        if (lane == 0) atomicExch(a.err, 1);
                        return;
                    }
                    __nanosleep(200);
                }
                __threadfence_block();
            }
            const int4 d = desc[it % kDescRing];
            const int l = d.x, i = d.y;
            ItemPos pos = {0, d.z, d.w};
            if (l < 0) {
                const int st = n % NST;
                if (!stage_free(n)) {
                    if (lane == 0) atomicExch(a.err, 1);
                    return;
                }
                if (lane == 0) mbar_arrive(&full_bar[st]);
                return;
            }
            const int sb0 = pos.sb * SB;
            const int sbw = min(SB, S - sb0);
            const size_t qrow = ((size_t)i * a.Lmax + l) * S + sb0;
            const int skip = a.front && pos.mt * TMB + TMB - 1 < a.front[(size_t)i * a.Lmax + (l - 1)];
            // this s-block's mem and time row, two strategies per lane (SB <= 64)
            const int mq0 = lane < sbw ? __ldg(a.mem_q + qrow + lane) : 0;
            const int mq1 = lane + 32 < sbw ? __ldg(a.mem_q + qrow + lane + 32) : 0;
            const int tq0 = lane < sbw ? __ldg(a.time_q + qrow + lane) : 0;
            const int tq1 = lane + 32 < sbw ? __ldg(a.time_q + qrow + lane + 32) : 0;
            for (int kc = 0; kc < NKC; ++kc, ++n) {
                const int st = n % NST;
                if (!stage_free(n)) {
                    if (lane == 0) atomicExch(a.err, 1);
                    return;
                }
                int32_t* meta = meta0 + st * META;
                if (kc == NKC - 1) {
                    if (lane < SB) { meta[lane] = mq0; meta[SB + lane] = tq0; }
                    if (lane + 32 < SB) { meta[lane + 32] = mq1; meta[SB + lane + 32] = tq1; }
                    if (lane == 0) meta[2 * SB] = i;
                }
                if (lane == 0) meta[2 * SB + 1] = skip;           // the consumers leave this chunk's k-steps out
                if (DOM && !P16 && lane < 2 * NMS) meta[2 * SB + 4 + lane] = 0;   // live rows: the consumers OR into these
                __syncwarp();
                if (lane == 0) mbar_arrive(&full_bar[st]);
            }
            if (pos.mt == 0) {
                // Cells no column maps to: m < mem(l,s), and the pad columns.
                if (MULTI && tile_done && !a.C) {
                    // rolling buffer: the cells still hold layer l-2, which layer l-1 may be reading
                    WaitClock wc;
                    while (ld_acquire_cta(&deps_ok) <= it) {
                        if (wc.expired()) {
                            if (lane == 0) atomicExch(a.err, 1);
                            return;
                        }
                        __nanosleep(100);
                    }
                }
                int32_t* out = a.C ? a.C + ((size_t)i * a.Lmax + l) * slice : a.roll + ((size_t)(l & 1) * a.B + i) * slice;
                uint8_t* aout = ARG ? a.A + ((size_t)i * a.Lmax + l) * slice : nullptr;
                for (int c = 0; c < sbw; ++c) {
                    const int mq = __shfl_sync(0xffffffffu, c < 32 ? mq0 : mq1, c & 31);
                    const int lo = min(mq, M + 1);
                    const size_t o = (size_t)(sb0 + c) * m_pitch;
                    for (int m = lane; m < lo + (m_pitch - M - 1); m += 32) {
                        const int mm = m < lo ? m : m - lo + M + 1;
                        out[o + mm] = kInf;
                        if (ARG) aout[o + mm] = 255;
                    }
                }
                if (MULTI && tile_done) {
                    // The tile is published only after these cells: the count goes to the store warp and
                    // on to the publisher by release / acquire in shared memory, and the publisher's fence
                    // is cumulative.  (A fence here would hold this warp, and with it the records of the
                    // next items, for thousands of cycles.)  A counter, not a barrier phase: this warp may
                    // be several first tiles ahead.
                    __syncwarp();
                    if (lane == 0) st_release_cta(&fill_count, ++nfilled);
                }
            }
        }
    }

    if (warp == NC + 2) {
        // ------------------------------------------------------------ store warp
        // Staging row `row` holds strategy sb0+row shifted by r = mem mod 4: staging column x is table
        // column g0 + x with g0 = m0 + mem - r a multiple of 4.  Columns r .. r+TMB-1 are real, and
        // table columns above M do not exist.  Each lane takes rows lane, lane+32: the 16-byte aligned
        // middle leaves as one bulk store, the few cells before and after it as plain stores.
        int it = 0;
        int nfill = 0;                                    // first tiles seen so far
        const bool publishing = MULTI && tile_done;
        // every way out tells the publisher (after the last hand-over, in program order)
        auto leave = [&](bool failed) {
            if (failed && lane == 0) atomicExch(a.err, 1);
            __syncwarp();
            if (lane == 0) *reinterpret_cast<volatile int*>(&store_exit) = 1;
        };
        for (;; ++it) {
            if (!mbar_wait_idle(&out_full, it & 1)) { leave(true); return; }
            // The consumers' staging writes (generic proxy) are ordered before this point by the barrier;
            // one proxy fence here makes them visible to the bulk stores below.  In the consumers it would
            // stall sixteen warps while the producer's loads are in flight.
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            const int4 d = desc[it % kDescRing];
            const int l = d.x, i = d.y;
            if (l < 0) break;                                     // no more items
            ItemPos pos = {0, d.z, d.w};
            const int m0 = pos.mt * TMB;
            const int sb0 = pos.sb * SB;
            const int sbw = min(SB, S - sb0);
            int32_t* out = (a.C ? a.C + ((size_t)i * a.Lmax + l) * slice : a.roll + ((size_t)(l & 1) * a.B + i) * slice)
                           + (size_t)sb0 * m_pitch;
            // store warp w takes rows w * RPW .. (w + 1) * RPW - 1 (with two warps: rows lane and lane + 32)
            for (int row = lane; row < (NSW <= 2 ? sbw : min(sbw, RPW)); row += (NSW <= 2 ? 32 * NSW : 32)) {
                const int mm = hdr0[row];
                const int r = mm & 3;
                const int g0 = m0 + mm - r;
                const int hi = min(r + TMB, M + 1 - g0);          // first staging column not to store
                if (hi <= r) continue;
                const int32_t* src = stg0 + row * RS;
                int32_t* dst = out + (size_t)row * m_pitch + (size_t)g0;
                const int lo4 = r ? 4 : 0, hi4 = hi & ~3;         // aligned middle [lo4, hi4)
                if (hi4 > lo4) bulk_s2g(dst + lo4, src + lo4, (uint32_t)(hi4 - lo4) * 4u);
                for (int x = r; x < min(lo4, hi); ++x) dst[x] = src[x];
                for (int x = max(hi4, lo4); x < hi; ++x) dst[x] = src[x];
            }
            bulk_commit();
            bulk_wait_read();                                     // the staging tile may be overwritten
            __syncwarp();
            if (lane == 0) red_release_cta_add(&out_drained, 1);
            if (publishing) {
                // Hand the item to the publisher warp once its stores are complete.  Making them visible
                // to the other SMs takes a fence, and a fence takes thousands of cycles while stores are
                // in flight: this warp must be back for the next tile sooner than that.
                if (pos.mt == 0) {                                // the helper's fill of this tile (it runs ahead)
                    ++nfill;
                    WaitClock wc;
                    while (ld_acquire_cta(&fill_count) < nfill) {
                        if (wc.expired()) { leave(true); return; }
                        __nanosleep(200);
                    }
                }
                bulk_wait_all();
                if (NSW > 1) {
                    WaitClock wc;                                 // the other store warp's rows are out as well
                    while (ld_acquire_cta(&drained_b) < (it + 1) * (NSW - 1)) {
                        if (wc.expired()) { leave(true); return; }
                        __nanosleep(100);
                    }
                }
                {
                    WaitClock wc;                                 // the publisher reads item records: keep it close
                    while (it + 1 - *reinterpret_cast<volatile int*>(&published_count) > kPublishLag) {
                        if (wc.expired()) { leave(true); return; }
                        __nanosleep(200);
                    }
                }
                __syncwarp();                                     // every lane's plain stores before lane 0's release
                if (lane == 0) st_release_cta(&drained_count, it + 1);
            }
        }
        bulk_wait_all();
        leave(false);
        return;
    }

    if (NSW > 1 && (NSW == 2 ? warp == NC + 4 : warp >= NC + 4)) {
        // ------------------------------------------------------------ further store warps (packed path)
        const int sw = warp - (NC + 4) + 1;
        for (int it = 0;; ++it) {
            if (!mbar_wait_idle(&out_full, it & 1)) {
                if (lane == 0) atomicExch(a.err, 1);
                return;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            const int4 d = desc[it % kDescRing];
            const int l = d.x, i = d.y;
            if (l < 0) return;
            const int m0 = d.z * TMB;
            const int sb0 = d.w * SB;
            const int sbw = min(SB, S - sb0);
            int32_t* out = (a.C ? a.C + ((size_t)i * a.Lmax + l) * slice : a.roll + ((size_t)(l & 1) * a.B + i) * slice)
                           + (size_t)sb0 * m_pitch;
            for (int row = (NSW == 2 ? lane + 32 : sw * RPW + lane); row < (NSW == 2 ? sbw : min(sbw, (sw + 1) * RPW)); row += (NSW == 2 ? 64 : 32)) {
                const int mm = hdr0[row];
                const int r = mm & 3;
                const int g0 = m0 + mm - r;
                const int hi = min(r + TMB, M + 1 - g0);
                if (hi <= r) continue;
                const int32_t* src = stg0 + row * RS;
                int32_t* dst = out + (size_t)row * m_pitch + (size_t)g0;
                const int lo4 = r ? 4 : 0, hi4 = hi & ~3;
                if (hi4 > lo4) bulk_s2g(dst + lo4, src + lo4, (uint32_t)(hi4 - lo4) * 4u);
                for (int x = r; x < min(lo4, hi); ++x) dst[x] = src[x];
                for (int x = max(hi4, lo4); x < hi; ++x) dst[x] = src[x];
            }
            bulk_commit();
            bulk_wait_read();
            __syncwarp();
            if (lane == 0) red_release_cta_add(&out_drained, 1);
            bulk_wait_all();
            __syncwarp();
            if (lane == 0) {
                if (NSW == 2) st_release_cta(&drained_b, it + 1);
                else red_release_cta_add(&drained_b, 1);
            }
        }
    }

    if (warp == NC + 3) {
        // ------------------------------------------------------------ publisher
        // Publishes finished tiles in a.tile_done: one proxy fence and one release fence for all the
        // items the store warp has handed over since the last round, then one relaxed add per item.
        // The hand-over (release / acquire in shared memory) puts the store warp's and the helper's
        // writes before the fence, which is cumulative.
        if (!(MULTI && tile_done)) return;
        int published = 0;
        for (;;) {
            int drained = 0, fin = 0;
            WaitClock wc;
            for (;;) {
                fin = *reinterpret_cast<volatile int*>(&store_exit);      // read before the count: then the count is final
                drained = ld_acquire_cta(&drained_count);
                if (drained > published || fin) break;
                if (wc.expired()) {
                    if (lane == 0) atomicExch(a.err, 1);
                    return;
                }
                __nanosleep(100);
            }
            if (drained == published) return;                     // the store warp has left and nothing is pending
            if (lane == 0) {
                asm volatile("fence.proxy.async;" ::: "memory");  // the data is read by other SMs' TMA loads
                __threadfence();
                for (int k = published; k < drained; ++k) {
                    const int4 d = desc[k % kDescRing];
                    red_relaxed_gpu_add(tile_done + (size_t)d.y * pl.ntiles_m + d.z, 1);
                }
                *reinterpret_cast<volatile int*>(&published_count) = drained;
            }
            __syncwarp();
            published = drained;
        }
    }

    // ---------------------------------------------------------------- consumers
    const int sg = warp % NSG, ms = warp / NSG;
    int acc[TM][TS];
    int arg[(ARG && !KEY) ? TM : 1][(ARG && !KEY) ? TS : 1];
    (void)arg;
    int n = 0, cst = 0;
    uint32_t cph = 0;
    // bounded wait until the store warp has read items 0 .. upto-1 out of the staging tile
    auto drained_wait = [&](int upto) -> bool {
        WaitClock wc;
        while (ld_acquire_cta(&out_drained) < upto * NSW)
            if (wc.expired()) return false;
        return true;
    };
    if constexpr (P16) {
        // ------------------------------------------------------------ consumers, packed 16-bit path
        constexpr int CW = (32 * TM + NSG - 1) / NSG;      // columns of the group each of its warps rebases
        constexpr int LPC = 16;                            // columns a warp handles at a time: two lanes per column,
                                                           // each with half of the rows (S / 2 <= 32 values, in registers)
        const int K = a.maxmem[1] + 1;                     // a candidate this far above the column's best cannot win
        // The ALU pipe is what limits this loop, the multiply-add pipe idles: the plain adds and shifts of the side
        // work (pack two values, split a result, put it back on its base) are written as multiply-adds with factors
        // the compiler cannot see through, so that they leave the ALU pipe to the add-mins.
        const uint32_t one = (uint32_t)(a.S != 0), two16 = one << 16;
        const int rows = S / 2;                            // S % 4 == 0: whole row pairs per lane
        constexpr bool dom = DOM;                          // leave dominated row pairs out (an instantiation of its own:
                                                           // the extra code costs the plain packed loop 4 %)
        for (int it = 0;; ++it) {
            const int st = it & 1;
            if (!mbar_wait(&full_bar[st], (it >> 1) & 1)) {
                if (lane == 0) atomicExch(a.err, 1);
                return;
            }
            const int4 d = desc[it % kDescRing];
            if (d.x < 0) {                                  // no more items: wake the store warp (once the previous item is out)
                if (!drained_wait(it)) {
                    if (lane == 0) atomicExch(a.err, 1);
                    return;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&out_full);
                return;
            }
            const int mw = d.z * TMB + ms * (32 * TM);      // first column of this warp
            const int nj = (mw > M) ? 0 : min(TM, (M - mw) / 32 + 1);
            int32_t* const stg = stage0 + st * stage_elems;
            uint32_t* const pkc = reinterpret_cast<uint32_t*>(stg);
            const uint32_t* const pkt = reinterpret_cast<const uint32_t*>(stg + Q * PP);
            int32_t* const basep = stg + Q * PP + Q * SB;
            uint32_t* const alivep = reinterpret_cast<uint32_t*>(basep + TMB);
            const int32_t* const meta = meta0 + st * META;
            const bool skipped = meta[2 * SB + 1] != 0;     // nothing but +inf to read: no data was loaded
            bool raw_released = false;
            if (!skipped) {
                // rebase: this warp's share of the group's columns, every row of them, read once
                const int cl = lane % LPC, h = lane / LPC;
                const int cend = min(sg * CW + CW, 32 * TM);
                const uint32_t kk = (uint32_t)K * 0x10001u;     // a pair of clamped values: neither row can win in this column
                uint32_t alive = 0;                             // row pairs of this lane's half that can still win in its columns
                for (int c0 = sg * CW; c0 < cend; c0 += LPC) {
                    const int cg = c0 + cl;                     // column inside the group
                    const int c = ms * (32 * TM) + min(cg, 32 * TM - 1);
                    const int32_t* rp = raw0 + (c / CB) * (S * PBOX) + (c % CB) + h * PBOX;    // rows h, h + 2, h + 4, ...
                    int v[32];
                    int mn = kInf;
                    if (rows == 32) {                           // S = 64: no row guards
#pragma unroll
                        for (int r = 0; r < 32; r += 2) {
                            v[r] = rp[(2 * r) * PBOX];
                            v[r + 1] = rp[(2 * r + 2) * PBOX];
                            mn = __vimin3_s32(mn, v[r], v[r + 1]);
                        }
                    } else {
#pragma unroll
                        for (int r = 0; r < 32; ++r) {
                            v[r] = r < rows ? rp[(2 * r) * PBOX] : kInf;
                            mn = min(mn, v[r]);
                        }
                    }
                    mn = min(mn, __shfl_xor_sync(0xffffffffu, mn, LPC));
                    if (dom && c0 + LPC >= cend) {
                        // last pass: every value this warp needs is in registers (the minimum has consumed them all),
                        // so the raw buffer goes back before the packing: with the inner loop this short the next
                        // tile's load latency is what the item waits for
                        raw_released = true;
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&empty_bar[0]);
                    }
                    if (cg < cend) {
                        uint32_t* out = pkc + h * PP + c;           // packed row 2q + h: rows 4q + h and 4q + 2 + h
                        // columns past the budget and columns without a finite value produce nothing
                        const bool track = dom && mn < kInf && mw + (c - ms * (32 * TM)) <= M;
#pragma unroll
                        for (int q = 0; q < 16; ++q)
                            if (rows == 32 || 2 * q < rows) {
                                const uint32_t d0 = (uint32_t)__viaddmin_s32(v[2 * q], -mn, K);
                                const uint32_t d1 = (uint32_t)__viaddmin_s32(v[2 * q + 1], -mn, K);
                                uint32_t pk;                                      // d0 | d1 << 16
                                asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(pk) : "r"(d1), "r"(two16), "r"(d0));
                                out[(2 * q) * PP] = pk;
                                if (track && pk != kk) alive |= 1u << (2 * q + h);
                            }
                        if (h == 0) basep[c] = mn;
                    }
                }
                if (dom) {
                    alive = __reduce_or_sync(0xffffffffu, alive);
                    if (lane == 0) alivep[ms * NSG + sg] = alive;
                }
            }
            __syncwarp();
            if (lane == 0) {
                if (!raw_released) mbar_arrive(&empty_bar[0]);   // this warp is done with the raw tile
                mbar_arrive(&conv_bar[ms]);                 // and its columns are there for the group
            }
            if (!mbar_wait(&conv_bar[ms], it & 1)) {
                if (lane == 0) atomicExch(a.err, 1);
                return;
            }
#pragma unroll
            for (int j = 0; j < TM; ++j)
#pragma unroll
                for (int u = 0; u < TS; ++u) acc[j][u] = -1;   // 0xffff in both halves
            if (!skipped && nj > 0) {
                const uint32_t* pc = pkc + ms * (32 * TM) + lane;
                const uint32_t* pt = pkt + sg * TS;
                int q = 0;
                auto steps = [&](auto ku) {
                    constexpr int KQ = decltype(ku)::value;
                    for (; q + KQ <= Q; q += KQ) {
#pragma unroll
                        for (int kk = 0; kk < KQ; ++kk) {
                            uint32_t c[TM];
#pragma unroll
                            for (int j = 0; j < TM; ++j) c[j] = pc[kk * PP + j * 32];
                            const uint4 t0 = *reinterpret_cast<const uint4*>(pt + kk * SB);
                            const uint4 t1 = *reinterpret_cast<const uint4*>(pt + kk * SB + 4);
                            const uint32_t t[TS] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w};
#pragma unroll
                            for (int j = 0; j < TM; ++j)
#pragma unroll
                                for (int u = 0; u < TS; ++u)
                                    acc[j][u] = (int)__viaddmin_u16x2(c[j], t[u], (uint32_t)acc[j][u]);
                        }
                        pc += KQ * PP;
                        pt += KQ * SB;
                    }
                };
                if (!dom) {
                    steps(std::integral_constant<int, 8>());
                    steps(std::integral_constant<int, 1>());
                } else {
                    // Dominated rows left out: a row pair whose values lie more than the largest transition entry
                    // above the column's best in every column of this group cannot supply a minimum (not even a
                    // tie), so only the pairs some warp of the group found alive are relaxed.  Same results.
                    uint32_t live = 0;
#pragma unroll
                    for (int g = 0; g < NSG; ++g) live |= alivep[ms * NSG + g];
                    while (live) {
                        const int qq = __ffs(live) - 1;
                        live &= live - 1;
                        uint32_t c[TM];
#pragma unroll
                        for (int j = 0; j < TM; ++j) c[j] = pc[qq * PP + j * 32];
                        const uint4 t0 = *reinterpret_cast<const uint4*>(pt + qq * SB);
                        const uint4 t1 = *reinterpret_cast<const uint4*>(pt + qq * SB + 4);
                        const uint32_t t[TS] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w};
#pragma unroll
                        for (int j = 0; j < TM; ++j)
#pragma unroll
                            for (int u = 0; u < TS; ++u)
                                acc[j][u] = (int)__viaddmin_u16x2(c[j], t[u], (uint32_t)acc[j][u]);
                    }
                }
            }
            int mm[TS], tt[TS];
            {
                const int4 m0v = *reinterpret_cast<const int4*>(meta + sg * TS);
                const int4 m1v = *reinterpret_cast<const int4*>(meta + sg * TS + 4);
                const int4 t0v = *reinterpret_cast<const int4*>(meta + SB + sg * TS);
                const int4 t1v = *reinterpret_cast<const int4*>(meta + SB + sg * TS + 4);
                mm[0] = m0v.x; mm[1] = m0v.y; mm[2] = m0v.z; mm[3] = m0v.w; mm[4] = m1v.x; mm[5] = m1v.y; mm[6] = m1v.z; mm[7] = m1v.w;
                tt[0] = t0v.x; tt[1] = t0v.y; tt[2] = t0v.z; tt[3] = t0v.w; tt[4] = t1v.x; tt[5] = t1v.y; tt[6] = t1v.z; tt[7] = t1v.w;
            }
            int bs[TM];
#pragma unroll
            for (int j = 0; j < TM; ++j) bs[j] = (skipped || j >= nj) ? kInf : basep[ms * (32 * TM) + j * 32 + lane];
            if (!drained_wait(it)) {                         // the previous item has been drained
                if (lane == 0) atomicExch(a.err, 1);
                return;
            }
            {
                const int s0l = sg * TS;
                const int col = ms * (32 * TM) + lane;
#pragma unroll
                for (int u = 0; u < TS; ++u) {
                    int32_t* R = stg0 + (s0l + u) * RS + (mm[u] & 3) + col;
#pragma unroll
                    for (int j = 0; j < TM; ++j)
                        if (j < nj) {
                            const uint32_t x = (uint32_t)acc[j][u];
                            uint32_t hi, v;
                            asm("mul.hi.u32 %0, %1, %2;" : "=r"(hi) : "r"(x), "r"(two16));     // x >> 16
                            const uint32_t w = __vminu2(x, hi);                     // the better of the two row parities (upper half: min with 0)
                            asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(v) : "r"(w), "r"(one), "r"((uint32_t)bs[j]));   // back on the column's base
                            R[j * 32] = (int)__viaddmin_u32(v, (uint32_t)tt[u], (uint32_t)kInf);   // +inf stays: below 2^32 unsigned
                        }
                }
                if (ms == 0) {
                    int v = mm[0];
#pragma unroll
                    for (int u = 1; u < TS; ++u) v = lane == u ? mm[u] : v;
                    if (lane < TS) hdr0[s0l + lane] = v;
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&out_full);            // release: the staging writes come before it
        }
    }
    const int kmax = (DOM && !P16) ? a.maxmem[1] : 0;      // largest transition entry (read once: a global load inside the loop waits behind the SM's stores)
    const int kmaxk = keyed ? a.maxmem[1] : 0;
    for (int it = 0;; ++it) {
        int l = 0, mw = 0, nj = 0;
        ItemPos pos = {0, 0, 0};
#pragma unroll
        for (int j = 0; j < TM; ++j)
#pragma unroll
            for (int u = 0; u < TS; ++u) {
                if (!KEY) acc[j][u] = keyed ? 0x7fffffff : kInf;       // min over candidates never exceeds kInf (keys: the largest key)
                if (ARGR) arg[ARGR ? j : 0][ARGR ? u : 0] = 255;
            }
        int mm[TS], tt[TS], inst = 0;
        int kbase[ARG ? TM : 1];                             // keyed argmin: the smallest previous-layer value of each of this lane's columns
        (void)kbase;
        for (int kc = 0; kc < NKC; ++kc, ++n) {
            const int st = cst;                             // = n % NST, phase cph = (n / NST) & 1
            if (!mbar_wait(&full_bar[st], cph)) {
                if (lane == 0) atomicExch(a.err, 1);
                return;
            }
            if (kc == 0) {
                // the item's record was posted before its first stage was filled
                const int4 d = desc[it % kDescRing];
                l = d.x;
                if (l < 0) {
                    // no more items: wake the store warp and leave.  Not before it has taken the previous
                    // item: two completions of out_full in a row would hide the first from its parity wait.
                    if (!drained_wait(it)) {
                        if (lane == 0) atomicExch(a.err, 1);
                        return;
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&out_full);
                    return;
                }
                pos.mt = d.z;
                pos.sb = d.w;
                mw = pos.mt * TMB + ms * (32 * TM);         // first column of this warp
                // 32-column groups of this warp that hold at least one column <= M
                nj = (mw > M) ? 0 : min(TM, (M - mw) / 32 + 1);
            }
            const int k0 = kc * KS;
            // nothing but +inf to read (see the producer): the accumulators stay at +inf
            const int kn = meta0[st * META + 2 * SB + 1] ? 0 : min(KS, S - k0);
            // this warp's columns inside their box, and its 8 trans columns
            const int32_t* cs = stage0 + st * stage_elems + ((ms * (32 * TM)) / BOXC) * (KS * BOXC) + (ms * (32 * TM)) % BOXC + lane;
            const int32_t* ts = stage0 + st * stage_elems + KS * TMB + sg * TS;
            bool keyed_done = false;
            if constexpr (ARG && !DOM && !P16) {
                if (keyed) {
                    keyed_done = true;
                    if constexpr (KEY) {
                        // The group's warps share the scan: each reads its share of the rows once (they stay in registers),
                        // posts the minima of those rows in its first row, reads everyone's after a barrier, and, after a
                        // second one (all have read the posted minima), writes its rows back as keys.  Three hand-overs an
                        // item, but a third of the shared-memory reads of a scan of all rows by every warp.
                        const int K = kmaxk + 1;
                        const int RW = (kn + NSG - 1) / NSG;            // <= TS rows a warp: the block holds at most NSG * TS
                        const int r0 = sg * RW, r1 = min(kn, r0 + RW);
                        int32_t* const cw = const_cast<int32_t*>(cs);
                        int v[TS][TM], pm[TM];
#pragma unroll
                        for (int j = 0; j < TM; ++j) pm[j] = kInf;
#pragma unroll
                        for (int rr = 0; rr < TS; ++rr)
#pragma unroll
                            for (int j = 0; j < TM; ++j) {
                                v[rr][j] = r0 + rr < r1 ? cs[(r0 + rr) * BOXC + j * 32] : kInf;
                                pm[j] = min(pm[j], v[rr][j]);
                            }
                        if (r0 < r1)
#pragma unroll
                            for (int j = 0; j < TM; ++j) cw[r0 * BOXC + j * 32] = pm[j];
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&conv_bar[ms]);
                        if (!mbar_wait(&conv_bar[ms], (3 * it) & 1)) {
                            if (lane == 0) atomicExch(a.err, 1);
                            return;
                        }
#pragma unroll
                        for (int j = 0; j < TM; ++j) kbase[ARG ? j : 0] = kInf;
                        for (int r = 0; r < kn; r += RW)
#pragma unroll
                            for (int j = 0; j < TM; ++j) kbase[ARG ? j : 0] = min(kbase[ARG ? j : 0], cs[r * BOXC + j * 32]);
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&conv_bar[ms]);
                        if (!mbar_wait(&conv_bar[ms], (3 * it + 1) & 1)) {
                            if (lane == 0) atomicExch(a.err, 1);
                            return;
                        }
                        // value -> key.  A candidate more than the largest transition entry above its column's best cannot
                        // win or tie, so the difference is capped there.
#pragma unroll
                        for (int rr = 0; rr < TS; ++rr)
                            if (r0 + rr < r1)
#pragma unroll
                                for (int j = 0; j < TM; ++j)
                                    cw[(r0 + rr) * BOXC + j * 32] = __viaddmin_s32(v[rr][j], -kbase[ARG ? j : 0], K) * 64 + (r0 + rr);
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&conv_bar[ms]);
                        if (!mbar_wait(&conv_bar[ms], (3 * it + 2) & 1)) {
                            if (lane == 0) atomicExch(a.err, 1);
                            return;
                        }
#pragma unroll
                        for (int j = 0; j < TM; ++j)
#pragma unroll
                            for (int u = 0; u < TS; ++u) acc[j][u] = 0x7fffffff;
                    } else {
                    // column minima of this warp's own columns over every row (each warp of the group scans them for itself:
                    // there is no room for a shared array of them beside the stages)
#pragma unroll
                    for (int j = 0; j < TM; ++j) kbase[ARG ? j : 0] = kInf;
                    for (int r = 0; r < kn; ++r)
#pragma unroll
                        for (int j = 0; j < TM; ++j) kbase[ARG ? j : 0] = min(kbase[ARG ? j : 0], cs[r * BOXC + j * 32]);
                    // every warp of the group has read the raw values before any of them is overwritten
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&conv_bar[ms]);
                    if (!mbar_wait(&conv_bar[ms], 0)) {                     // two phases of this barrier per item: scan done, keys written
                        if (lane == 0) atomicExch(a.err, 1);
                        return;
                    }
                    if (kn > 0) {
                        // this warp's share of the rows, all columns of the group: value -> key.  A candidate more than the
                        // largest transition entry above its column's best cannot win or tie, so the difference is capped there.
                        const int K = kmaxk + 1;
                        int32_t* const cw = const_cast<int32_t*>(cs);
                        const int RW = (kn + NSG - 1) / NSG;
                        for (int r = sg * RW; r < min(kn, sg * RW + RW); ++r)
#pragma unroll
                            for (int j = 0; j < TM; ++j) {
                                const int d = __viaddmin_s32(cw[r * BOXC + j * 32], -kbase[ARG ? j : 0], K);
                                cw[r * BOXC + j * 32] = d * 64 + r;
                            }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&conv_bar[ms]);
                    if (!mbar_wait(&conv_bar[ms], 1)) {
                        if (lane == 0) atomicExch(a.err, 1);
                        return;
                    }
                    }
                    if (nj > 0) {
                        int k = 0;
                        auto ksteps = [&](auto ku) {
                            constexpr int K = decltype(ku)::value;
                            for (; k + K <= kn; k += K) {
#pragma unroll
                                for (int kk = 0; kk < K; ++kk) {
                                    int c[TM];
#pragma unroll
                                    for (int j = 0; j < TM; ++j) c[j] = cs[kk * BOXC + j * 32];
                                    const int4 t0 = *reinterpret_cast<const int4*>(ts + kk * SB);
                                    const int4 t1 = *reinterpret_cast<const int4*>(ts + kk * SB + 4);
                                    const int t[TS] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w};
#pragma unroll
                                    for (int j = 0; j < TM; ++j)
#pragma unroll
                                        for (int u = 0; u < TS; ++u) acc[j][u] = __viaddmin_s32(c[j], t[u], acc[j][u]);
                                }
                                cs += K * BOXC;
                                ts += K * SB;
                            }
                        };
                        ksteps(std::integral_constant<int, 16>());
                        ksteps(std::integral_constant<int, 4>());
                        ksteps(std::integral_constant<int, 1>());
                        // key -> (cost before time(l,s), row): what the epilogue expects of the plain loop
                        // (the keys-only instantiation splits them in its epilogue)
                        if constexpr (!KEY)
#pragma unroll
                        for (int j = 0; j < TM; ++j)
#pragma unroll
                            for (int u = 0; u < TS; ++u) {
                                const int key = acc[j][u];
                                arg[ARGR ? j : 0][ARGR ? u : 0] = key & 63;
                                acc[j][u] = kbase[ARG ? j : 0] >= kInf ? kInf : kbase[ARG ? j : 0] + (key >> 6);
                            }
                    }
                    // the stage was rewritten by plain stores; the next load into it comes through the async proxy
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                }
            }
            if constexpr (KEY) {
            } else if (keyed_done) {
            } else if constexpr (DOM && !P16) {
                // Dominated rows left out (one chunk per item, S <= 64: the host takes this instantiation only then).
                // A candidate more than the largest transition entry above its column's best cannot win or tie;
                // a row that is such in every column of this group's tile is not relaxed.  Each warp scans its
                // share of the group's columns (minimum, then one compare per value), the group ORs the rows still
                // alive into two words beside the item's record, and after a barrier walks their set bits.
                uint32_t* const live_w = reinterpret_cast<uint32_t*>(meta0 + st * META + 2 * SB + 4 + 2 * ms);
                if (kn > 0) {
                    constexpr int CW = (32 * TM + NSG - 1) / NSG;   // columns of the group each of its warps scans
                    const int cend = min(sg * CW + CW, 32 * TM);
                    uint32_t lo = 0, hi = 0;
                    for (int c0 = sg * CW; c0 < cend; c0 += 32) {
                        const int cg = c0 + lane;
                        const int c = ms * (32 * TM) + min(cg, 32 * TM - 1);
                        const int32_t* p = stage0 + st * stage_elems + (c / BOXC) * (KS * BOXC) + c % BOXC;
                        int mn = kInf;
#pragma unroll 4
                        for (int r = 0; r < kn; ++r) mn = min(mn, p[r * BOXC]);
                        // columns past the budget and columns without a finite value produce nothing
                        if (cg < cend && mn < kInf && mw + cg <= M) {
                            const int lim = mn + kmax;              // both below 2^30
#pragma unroll 4
                            for (int r = 0; r < min(kn, 32); ++r) lo |= (p[r * BOXC] <= lim) ? 1u << r : 0u;
#pragma unroll 4
                            for (int r = 32; r < kn; ++r) hi |= (p[r * BOXC] <= lim) ? 1u << (r - 32) : 0u;
                        }
                    }
                    lo = __reduce_or_sync(0xffffffffu, lo);
                    hi = __reduce_or_sync(0xffffffffu, hi);
                    if (lane == 0) {
                        if (lo) atomicOr(live_w, lo);
                        if (hi) atomicOr(live_w + 1, hi);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&conv_bar[ms]);
                if (!mbar_wait(&conv_bar[ms], it & 1)) {
                    if (lane == 0) atomicExch(a.err, 1);
                    return;
                }
                if (nj > 0 && kn > 0) {
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        uint32_t lv = *reinterpret_cast<volatile uint32_t*>(live_w + half);
                        while (lv) {
                            const int r = __ffs(lv) - 1 + 32 * half;
                            lv &= lv - 1;
                            int c[TM];
#pragma unroll
                            for (int j = 0; j < TM; ++j) c[j] = cs[r * BOXC + j * 32];
                            const int4 t0 = *reinterpret_cast<const int4*>(ts + r * SB);
                            const int4 t1 = *reinterpret_cast<const int4*>(ts + r * SB + 4);
                            const int t[TS] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w};
#pragma unroll
                            for (int j = 0; j < TM; ++j)
#pragma unroll
                                for (int u = 0; u < TS; ++u) {
                                    if (ARG) {                  // rows come in ascending order: the lowest row wins a tie
                                        const int cand = c[j] + t[u];
                                        if (cand < acc[j][u]) { acc[j][u] = cand; arg[ARGR ? j : 0][ARGR ? u : 0] = r; }
                                    } else {
                                        acc[j][u] = __viaddmin_s32(c[j], t[u], acc[j][u]);
                                    }
                                }
                        }
                    }
                }
            } else {
                if (nj == TM) {
                    // trips of KU k-steps, then of 4, then single ones: loop control and pointer bumps are ALU
                    // instructions too, one trip of 16 k-steps spends 4 of them on 512 relaxations
                    int k = 0;
                    auto steps = [&](auto ku) {
                        constexpr int K = decltype(ku)::value;
                        for (; k + K <= kn; k += K) {
    #pragma unroll
                            for (int kk = 0; kk < K; ++kk) {
                                int c[TM];
    #pragma unroll
                                for (int j = 0; j < TM; ++j) c[j] = cs[kk * BOXC + j * 32];
                                const int4 t0 = *reinterpret_cast<const int4*>(ts + kk * SB);
                                const int4 t1 = *reinterpret_cast<const int4*>(ts + kk * SB + 4);
                                const int t[TS] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w};
    #pragma unroll
                                for (int j = 0; j < TM; ++j)
    #pragma unroll
                                    for (int u = 0; u < TS; ++u) {
                                        if (ARG) {
                                            const int cand = c[j] + t[u];
                                            if (cand < acc[j][u]) { acc[j][u] = cand; arg[ARGR ? j : 0][ARGR ? u : 0] = k0 + k + kk; }
                                        } else {
                                            acc[j][u] = __viaddmin_s32(c[j], t[u], acc[j][u]);
                                        }
                                    }
                            }
                            cs += K * BOXC;
                            ts += K * SB;
                        }
                    };
                    steps(std::integral_constant<int, KU>());
                    steps(std::integral_constant<int, 4>());
                    steps(std::integral_constant<int, 1>());
                } else if (nj > 0) {
                    // ragged last tile: only the first nj column groups carry work
                    for (int k = 0; k < kn; ++k) {
                        const int4 t0 = *reinterpret_cast<const int4*>(ts + k * SB);
                        const int4 t1 = *reinterpret_cast<const int4*>(ts + k * SB + 4);
                        const int t[TS] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w};
    #pragma unroll
                        for (int j = 0; j < TM; ++j)
                            if (j < nj) {
                                const int c = cs[k * BOXC + j * 32];
    #pragma unroll
                                for (int u = 0; u < TS; ++u) {
                                    const int cand = c + t[u];
                                    if (cand < acc[j][u]) { acc[j][u] = cand; if (ARG) arg[ARGR ? j : 0][ARGR ? u : 0] = k0 + k; }
                                }
                            }
                    }
                }
            }
            if (kc == NKC - 1) {
                // the item's record must be read before the stage is handed back
                const int32_t* meta = meta0 + st * META;
                const int4 m0v = *reinterpret_cast<const int4*>(meta + sg * TS);
                const int4 m1v = *reinterpret_cast<const int4*>(meta + sg * TS + 4);
                const int4 t0v = *reinterpret_cast<const int4*>(meta + SB + sg * TS);
                const int4 t1v = *reinterpret_cast<const int4*>(meta + SB + sg * TS + 4);
                mm[0] = m0v.x; mm[1] = m0v.y; mm[2] = m0v.z; mm[3] = m0v.w; mm[4] = m1v.x; mm[5] = m1v.y; mm[6] = m1v.z; mm[7] = m1v.w;
                tt[0] = t0v.x; tt[1] = t0v.y; tt[2] = t0v.z; tt[3] = t0v.w; tt[4] = t1v.x; tt[5] = t1v.y; tt[6] = t1v.z; tt[7] = t1v.w;
                inst = meta[2 * SB];
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty_bar[st]);      // this warp is done reading the stage
            if (++cst == NST) { cst = 0; cph ^= 1; }
        }

        // Epilogue: add time(l,s) and hand the tile to the store warps through the staging tile;
        // row s is written shifted by mem(l,s) mod 4 (see the store warps).
        if (!drained_wait(it)) {                             // the previous item has been drained
            if (lane == 0) atomicExch(a.err, 1);
            return;
        }
        {
            const int s0l = sg * TS;                          // first strategy of this warp inside the block
            const int col = ms * (32 * TM) + lane;
#pragma unroll
            for (int u = 0; u < TS; ++u) {
                int32_t* R = stg0 + (s0l + u) * RS + (mm[u] & 3) + col;
                // finite sums stay below kInf and acc <= kInf, so acc + time cannot wrap
#pragma unroll
                for (int j = 0; j < TM; ++j)
                    if (j < nj) {
                        if constexpr (KEY) {
                            // key = (difference to the column's smallest value) << 6 | row; a column without a finite
                            // value has base +inf and stays +inf (base + 2^25 does not wrap)
                            const int v = __viaddmin_s32(kbase[ARG ? j : 0], acc[j][u] >> 6, kInf);
                            acc[j][u] = v >= kInf ? 255 : (acc[j][u] & 63);      // what the argmin table gets
                            R[j * 32] = __viaddmin_s32(v, tt[u], kInf);
                        } else {
                            R[j * 32] = __viaddmin_s32(acc[j][u], tt[u], kInf);
                        }
                    }
            }
            if (ms == 0) {
                // lane u posts mem of strategy u: selects and one store (eight divergent stores cost a thousand cycles)
                int v = mm[0];
#pragma unroll
                for (int u = 1; u < TS; ++u) v = lane == u ? mm[u] : v;
                if (lane < TS) hdr0[s0l + lane] = v;
            }
            if (ARG && nj > 0) {
                const int s0 = pos.sb * SB + s0l;
                const int base = M - mw - lane;
#pragma unroll
                for (int u = 0; u < TS; ++u)
                    if (s0 + u < S) {
                        const int lim = base - mm[u];
                        uint8_t* pa = a.A + ((size_t)inst * a.Lmax + l) * slice + (size_t)(s0 + u) * m_pitch + (size_t)(mm[u] + mw + lane);
#pragma unroll
                        for (int j = 0; j < TM; ++j)
                            if (j * 32 <= lim) pa[j * 32] = KEY ? (uint8_t)acc[j][u] : (uint8_t)(acc[j][u] >= kInf ? 255 : arg[ARGR ? j : 0][ARGR ? u : 0]);
                    }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&out_full);                // release: the staging writes come before it
    }
}

// C_last[i] = layer L[i]-1 of instance i (from the full table, or from the rolling buffer that
// layer was written to), 128 bits per thread.
__global__ void copy_last_kernel(DpArgs a)
{
    const int i = blockIdx.y;
    if (a.status[i] != 0) return;
    const int Li = a.L[i];
    const size_t slice = (size_t)a.S * a.m_pitch;
    const int32_t* src = a.C ? a.C + ((size_t)i * a.Lmax + (Li - 1)) * slice : a.roll + ((size_t)((Li - 1) & 1) * a.B + i) * slice;
    const int4* s4 = reinterpret_cast<const int4*>(src);
    int4* d4 = reinterpret_cast<int4*>(a.C_last + (size_t)i * slice);
    for (size_t k = (size_t)blockIdx.x * blockDim.x + threadIdx.x; k < slice / 4; k += (size_t)gridDim.x * blockDim.x) d4[k] = s4[k];
}

// Sets the TIMEOUT bit everywhere when a bounded wait ran out.
__global__ void finalize_kernel(int B, const int32_t* err, int32_t* status)
{
    if (*err == 0) return;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < B; i += gridDim.x * blockDim.x)
        status[i] |= GALV_STATUS_TIMEOUT;
}

// maps == nullptr: only opt the instantiation into its dynamic shared memory.  Layers l_first..l_last-1;
// more than one layer means the CTAs wait on one another's tiles, so the launch is cooperative
// (all CTAs guaranteed co-resident).
template <int TM, int NSG, int NMS, bool ARG>
cudaError_t launch_one(const DpArgs& a, const DpPlan& pl, int l_first, int l_last, cudaStream_t st, const CUtensorMap* maps,
                       bool packed)
{
    auto kern = layer_tiled_kernel<TM, NSG, NMS, ARG, false>;
    auto kern_dom = layer_tiled_kernel<TM, NSG, NMS, ARG, false, false, true>;
    auto kern_multi = layer_tiled_kernel<TM, NSG, NMS, false, true>;
    auto kern_packed = layer_tiled_kernel<TM, NSG, NMS, false, true, true>;
    auto kern_packed_dom = layer_tiled_kernel<TM, NSG, NMS, false, true, true, true>;
    auto kern_multi_dom = layer_tiled_kernel<TM, NSG, NMS, false, true, false, true>;
    auto kern_multi_key = layer_tiled_kernel<TM, NSG, NMS, true, true, false, false, true>;
    if (!maps) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.smem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(kern_dom, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.smem);
        if (e == cudaSuccess && !ARG) e = cudaFuncSetAttribute(kern_multi, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.smem);
        if (e == cudaSuccess && !ARG) e = cudaFuncSetAttribute(kern_packed, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.smem);
        if (e == cudaSuccess && !ARG) e = cudaFuncSetAttribute(kern_packed_dom, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.smem);
        if (e == cudaSuccess && !ARG) e = cudaFuncSetAttribute(kern_multi_dom, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.smem);
        if (e == cudaSuccess && ARG) e = cudaFuncSetAttribute(kern_multi_key, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.smem);
        return e;
    }
    if (packed) {
        // the packed 16-bit kernel over all layers: its own tensor maps (whole-tile boxes, packed trans rows)
        void* args[] = {(void*)&a, (void*)&pl, (void*)&l_first, (void*)&l_last, (void*)&maps[2], (void*)&maps[3]};
        return cudaLaunchCooperativeKernel(a.skip_dom ? (const void*)kern_packed_dom : (const void*)kern_packed, dim3(pl.grid), dim3((NSG * NMS + (a.skip_dom ? 7 : 5)) * 32), args, (size_t)pl.p16_smem, st);
    }
    if (l_last - l_first > 1) {
        void* args[] = {(void*)&a, (void*)&pl, (void*)&l_first, (void*)&l_last, (void*)&maps[0], (void*)&maps[1]};
        if (ARG)     // argmin table through keys, all layers in one launch
            return cudaLaunchCooperativeKernel((const void*)kern_multi_key, dim3(pl.grid), dim3((NSG * NMS + 4) * 32), args, (size_t)pl.smem, st);
        // dominated rows are left out where all S <= 64 rows of a tile sit in one stage
        const bool dom = a.skip_dom && pl.nkc == 1 && a.S <= 64;
        return cudaLaunchCooperativeKernel(dom ? (const void*)kern_multi_dom : (const void*)kern_multi, dim3(pl.grid), dim3((NSG * NMS + 4) * 32), args, (size_t)pl.smem, st);
    }
    if (a.skip_dom && pl.nkc == 1 && a.S <= 64)
        kern_dom<<<pl.grid, (NSG * NMS + 4) * 32, pl.smem, st>>>(a, pl, l_first, l_last, maps[0], maps[1]);
    else
        kern<<<pl.grid, (NSG * NMS + 4) * 32, pl.smem, st>>>(a, pl, l_first, l_last, maps[0], maps[1]);
    return cudaGetLastError();
}

// nsg warps along s, 16/nsg (rounded down) along m: one instantiation per s-block width.
template <bool ARG>
cudaError_t launch_tiled(const DpArgs& a, const DpPlan& pl, int l_first, int l_last, cudaStream_t st, const CUtensorMap* maps,
                         bool packed = false)
{
    switch (pl.nsg) {
    case 1: return launch_one<4, 1, 16, ARG>(a, pl, l_first, l_last, st, maps, packed);
    case 2: return launch_one<4, 2, 8, ARG>(a, pl, l_first, l_last, st, maps, packed);
    case 3: return launch_one<4, 3, 5, ARG>(a, pl, l_first, l_last, st, maps, packed);
    case 4: return launch_one<4, 4, 4, ARG>(a, pl, l_first, l_last, st, maps, packed);
    case 5: return launch_one<4, 5, 3, ARG>(a, pl, l_first, l_last, st, maps, packed);
    case 6: return launch_one<4, 6, 2, ARG>(a, pl, l_first, l_last, st, maps, packed);
    case 7: return launch_one<4, 7, 2, ARG>(a, pl, l_first, l_last, st, maps, packed);
    case 8: return launch_one<4, 8, 2, ARG>(a, pl, l_first, l_last, st, maps, packed);
    default: return cudaErrorInvalidConfiguration;
    }
}

}  // namespace

// ---------------------------------------------------------------- host side

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

typedef CUresult (*PFN_encodeTiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                    const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

WsLayout galv_ws_layout(const galv_shape* sh)
{
    WsLayout w;
    size_t off = 0;
    w.order = off;   off = align256(off + (size_t)sh->B * 4);
    w.nactive = off; off = align256(off + (size_t)(sh->Lmax + 1) * 4);
    w.scratch = off; off = align256(off + (size_t)4 * (sh->Lmax + 2) * 4);    // two int32 arrays, one 64-bit array
    w.err = off;     off = align256(off + 32);                 // error flag, largest mem, largest trans, path chosen, keyed argmin
    w.minmem_l = off; off = align256(off + (size_t)(sh->Lmax + 1) * 4);
    w.ntiles = off;   off = align256(off + (size_t)(sh->Lmax + 1) * 4);
    w.istart = off;   off = align256(off + (size_t)(sh->Lmax + 1) * 8);
    w.tcount = off;   off = align256(off + (size_t)sh->Lmax * ((sh->M + 128) / 128) * 4);
    w.front = off;    off = align256(off + (size_t)sh->B * sh->Lmax * 4);
    w.tile_done = off; off = align256(off + (size_t)sh->B * ((sh->M + 128) / 128) * 4);   // per (instance, tile of >= 128 columns)
    w.trans_p = off;                                           // packed trans rows for the 16-bit path (S <= 64, S % 4 == 0)
    if (sh->S <= 64 && sh->S % 4 == 0 && !(sh->flags & (GALV_KERNEL_NO_PACKED | GALV_STORE_ARGMIN | GALV_KERNEL_PER_LAYER | GALV_KERNEL_REFERENCE)))
        off = align256(off + (size_t)sh->B * ((sh->flags & GALV_TRANS_PER_LAYER) ? sh->Lmax : 1) * (sh->S / 2) * sh->S * 4);
    else if (sh->S <= 64 && (sh->flags & GALV_STORE_ARGMIN) && !(sh->flags & GALV_KERNEL_REFERENCE))
        off = align256(off + (size_t)sh->B * ((sh->flags & GALV_TRANS_PER_LAYER) ? sh->Lmax : 1) * sh->S * sh->S * 4);   // shifted copy for the keyed argmin loop
    w.roll = off;
    if (!(sh->flags & GALV_STORE_C_FULL)) off = align256(off + (size_t)2 * sh->B * sh->S * sh->m_pitch * 4);
    w.total = off;
    return w;
}

bool galv_dp_make_plan(const galv_ctx* ctx, const galv_shape* sh, DpPlan* pl)
{
    const int S = sh->S;
    const int spad = (S + TS - 1) / TS * TS;
    pl->tm = 4;
    pl->nsb = (spad + 63) / 64;
    pl->sb = ((S + pl->nsb - 1) / pl->nsb + TS - 1) / TS * TS;
    pl->nsg = pl->sb / TS;
    pl->nms = 16 / pl->nsg;
    if (pl->nms < 1) pl->nms = 1;
    pl->tmb = pl->nms * 32 * pl->tm;
    pl->threads = (pl->nsg * pl->nms + 4) * 32;           // consumer warps + producer, helper, store and publisher warps
    // stages of ks * (tmb + sb) ints: aim at <= 40 KB each, 2..4 of them in the opt-in shared memory
    const int staging = (pl->sb * (pl->tmb + 4) + pl->sb) * 4;              // staging tile and its header
    const int budget = ctx->smem_optin - kStaticSmemReserve;               // dynamic shared memory a CTA may have
    const int row = (pl->tmb + pl->sb) * 4;
    // chunks of s': as few per item as leave room for two stages (every chunk costs the consumers
    // a barrier hand-over), of equal size, multiples of 8 rows; then as many stages as fit
    const int dom_words = (sh->flags & GALV_SKIP_DOMINATED) ? ((2 * pl->nms + 3) & ~3) : 0;   // live-row words per column group in each item record
    int nkc = 1, ks = S, stage_bytes = 0, nst = 0, extra = 0;
    for (;; ++nkc) {
        ks = (S + nkc - 1) / nkc;
        if (ks >= 8) ks = (ks + 7) & ~7;
        stage_bytes = (ks * row + 127) & ~127;
        for (nst = kMaxStages; nst >= 2; --nst) {
            extra = ((nst * (2 * pl->sb + 4 + dom_words) + 31) & ~31) * 4 + staging;  // item records of the stages
            if (nst * stage_bytes + extra <= budget) break;
        }
        if (nst >= 2 || ks == 1) break;
    }
    if (nst < 2) return false;
    pl->ks = ks;
    pl->nst = nst;
    pl->nkc = (S + ks - 1) / ks;
    pl->ntiles_m = (sh->M + 1 + pl->tmb - 1) / pl->tmb;
    pl->smem = nst * stage_bytes + extra;
    pl->tma_t = (S % 4) == 0;                             // trans row pitch a multiple of 16 bytes
    // Packed 16-bit path: the whole previous-layer tile (all S rows, one buffer) as it comes from the table, two
    // stages of its packed form (row pairs), the packed trans rows and the column bases; no argmin table.
    {
        const int q = S / 2;
        const int raw = (S * 144 * (pl->tmb / 128) * 4 + 127) & ~127;       // boxes of 128 + 16 columns
        const int pst = ((q * (pl->tmb + 16) + q * pl->sb + pl->tmb + pl->nsg * pl->nms) * 4 + 127) & ~127;
        const int total = raw + 2 * pst + ((2 * (2 * pl->sb + 4) + 31) & ~31) * 4 + staging;
        pl->p16 = S <= 64 && S % 4 == 0 && pl->nsb == 1 && !(sh->flags & GALV_STORE_ARGMIN) && total <= budget;
        pl->p16_smem = total;
    }
    const long long items = (long long)sh->B * pl->ntiles_m * pl->nsb;
    pl->grid = (int)(items < ctx->num_sms ? items : ctx->num_sms);
    return true;
}

// Tensor map of a row-major int32 matrix [rows][cols] (row pitch = cols * 4 bytes) with a dense box.
static cudaError_t encode_2d(CUtensorMap* map, void* base, size_t cols, size_t rows, int box_cols, int box_rows)
{
    static PFN_encodeTiled fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
        if (e != cudaSuccess) return e;
        if (q != cudaDriverEntryPointSuccess || !p) return cudaErrorNotSupported;
        fn = reinterpret_cast<PFN_encodeTiled>(p);
    }
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 4};
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_INT32, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

cudaError_t galv_dp_configure(const galv_ctx* ctx)
{
    // opt every instantiation into the large dynamic shared memory once per context
    DpArgs a{};
    DpPlan pl{};
    pl.smem = ctx->smem_optin - kStaticSmemReserve;
    for (int nsg = 1; nsg <= 8; ++nsg) {
        pl.nsg = nsg;
        cudaError_t e = launch_tiled<false>(a, pl, 0, 0, nullptr, nullptr);
        if (e == cudaSuccess) e = launch_tiled<true>(a, pl, 0, 0, nullptr, nullptr);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t galv_dp_launch(galv_ctx* ctx, const galv_shape* sh, const DpArgs& a, cudaStream_t st)
{
    cudaError_t e;
    const int B = a.B, Lmax = a.Lmax, S = a.S;
    {
        // Small batches: one cluster per instance, the whole search in one launch (no workspace but the path flag).
        ClPlan cp;
        if (galv_cluster_plan(ctx, sh, &cp)) {
            e = galv_cluster_launch(ctx, sh, cp, a, st);
            if (e == cudaSuccess) return e;
            (void)cudaGetLastError();                        // the clusters cannot be placed on this device right now: tiled kernels
        }
    }
    e = cudaMemsetAsync(a.scratch, 0, (size_t)4 * (Lmax + 2) * 4, st);      // histogram, fill and work counters
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(a.err, 0, 32, st);                       // error flag, largest mem, largest trans, path, keyed
    if (e != cudaSuccess) return e;
    const bool reference = (sh->flags & GALV_KERNEL_REFERENCE) != 0;
    DpPlan pl;
    std::memset(&pl, 0, sizeof(pl));
    if (!reference && !galv_dp_make_plan(ctx, sh, &pl)) return cudaErrorInvalidConfiguration;
    if (reference) { pl.tmb = 256; pl.ntiles_m = (a.M + 256) / 256; }
    e = cudaMemsetAsync(a.minmem_l, 0x7f, (size_t)(Lmax + 1) * 4, st);
    if (e != cudaSuccess) return e;
    // All layers in one cooperative launch when the grid's CTAs can be co-resident (they wait on one
    // another's tiles); with an argmin table whose loop cannot work on keys, on request, or for the reference
    // kernel: one launch per layer.
    // With the two-layer rolling buffer an item also waits for the readers of the cells it overwrites.
    const bool persistent = !reference && !a.A && Lmax > 2 && !(sh->flags & GALV_KERNEL_PER_LAYER);
    // The packed 16-bit kernel is launched as well when the shape allows it; which of the two runs is decided on
    // the device, where the largest transition entry is known (the other one returns at once).
    const int will_p16 = persistent && pl.p16 && !(sh->flags & GALV_KERNEL_NO_PACKED);
    validate_kernel<<<B, 128, 0, st>>>(B, Lmax, S, a.M, (long long)a.trans_layer, a.L, a.time_q, a.mem_q, a.trans_q, a.status, a.err + 1, a.minmem_l,
                                       (sh->flags & GALV_SKIP_INFEASIBLE) ? a.front : nullptr);
    schedule_kernel<<<1, 1024, 0, st>>>(B, Lmax, a.M, pl.tmb, pl.ntiles_m, pl.nsb, a.L, a.status, a.order, a.nactive, a.scratch,
                                         a.minmem_l, a.ntiles, a.istart, a.tcount, will_p16, a.err + 1);
    auto base_layer = [&]() {
        int gx = (a.m_pitch + 255) / 256;
        if (gx > 8) gx = 8;
        for (int b0 = 0; b0 < B; b0 += 65535) {           // grid.z limit
            DpArgs s = a;
            const int nb = (B - b0 < 65535) ? B - b0 : 65535;
            s.L += b0; s.status += b0;
            s.time_q += (size_t)b0 * Lmax * S; s.mem_q += (size_t)b0 * Lmax * S;
            if (s.C) s.C += (size_t)b0 * Lmax * S * a.m_pitch;
            if (s.A) s.A += (size_t)b0 * Lmax * S * a.m_pitch;
            s.C_last += (size_t)b0 * S * a.m_pitch;
            s.roll += (size_t)b0 * S * a.m_pitch;
            base_layer_kernel<<<dim3(gx, S, nb), 256, 0, st>>>(s);
        }
    };
    base_layer();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;

    CUtensorMap maps[4];
    std::memset(maps, 0, sizeof(maps));
    bool keyed_possible = false;
    if (!reference) {
        // previous-layer values as a 2-D tensor [rows of m_pitch columns]; box = ks rows x (<=256) columns
        const int boxc = 32 * pl.tm * ((pl.nms % 2 == 0 && 64 * pl.tm <= 256) ? 2 : 1);
        const size_t rows = a.C ? (size_t)B * Lmax * S : (size_t)2 * B * S;
        if ((e = encode_2d(&maps[0], a.C ? (void*)a.C : (void*)a.roll, (size_t)a.m_pitch, rows, boxc, pl.ks)) != cudaSuccess) return e;
        // argmin table with keys: the layer kernels read the shifted copy of the transition matrices
        // (not with GALV_SKIP_DOMINATED: that instantiation walks the live rows with the plain loop)
        keyed_possible = a.A != nullptr && S <= 64 && pl.nkc == 1 && pl.nsb == 1 && !(sh->flags & GALV_SKIP_DOMINATED);
        if (keyed_possible) {
            const long long n = (long long)B * (a.trans_layer ? Lmax : 1) * S * S;
            long long blocks = (n + 255) / 256;
            if (blocks > 148 * 8) blocks = 148 * 8;
            key_trans_kernel<<<(int)blocks, 256, 0, st>>>(n, a.trans_q, a.trans_k, a.err + 1);
        }
        if (pl.tma_t &&
            (e = encode_2d(&maps[1], keyed_possible ? (void*)a.trans_k : (void*)a.trans_q, (size_t)S, (size_t)B * (a.trans_layer ? Lmax : 1) * S, pl.sb, pl.ks)) != cudaSuccess) return e;
        if (will_p16) {
            // whole tiles (all S rows) of the previous layer; packed trans rows [S/2 row pairs][S]
            const long long n_mats = (long long)B * (a.trans_layer ? Lmax : 1);
            if ((e = encode_2d(&maps[2], a.C ? (void*)a.C : (void*)a.roll, (size_t)a.m_pitch, rows, 144, S)) != cudaSuccess) return e;
            if ((e = encode_2d(&maps[3], (void*)a.trans_p, (size_t)S, (size_t)n_mats * (S / 2), pl.sb, S / 2)) != cudaSuccess) return e;
            long long blocks = (n_mats * (S / 2) * S + 255) / 256;
            if (blocks > 148 * 8) blocks = 148 * 8;
            pack_trans_kernel<<<(int)blocks, 256, 0, st>>>(n_mats, S, a.trans_q, a.trans_p);
        }
    }
    DpArgs ap = a;
    ap.withhold = (sh->flags & GALV_DEBUG_WITHHOLD_LOAD) != 0;
    ap.skip_dom = (sh->flags & GALV_SKIP_DOMINATED) != 0;
    ap.keyed = keyed_possible;
    if (!(sh->flags & GALV_SKIP_INFEASIBLE)) ap.front = nullptr;
    ap.tile_done = nullptr;
    ap.maxmem = a.err + 1;
    ap.keyed_multi = 0;
    // Argmin table where keys are possible: one cooperative launch over all layers (it returns at once when the device
    // finds the transition entries too large for keys), then the launches per layer, which return at once when it ran.
    const bool key_multi = keyed_possible && Lmax > 2 && !(sh->flags & GALV_KERNEL_PER_LAYER);
    if (persistent || key_multi) {
        ap.tile_done = a.tile_done;
        if ((e = cudaMemsetAsync(a.tile_done, 0, (size_t)B * pl.ntiles_m * 4, st)) != cudaSuccess) return e;
    }
    const int pk = ctx->prof_count % 64;
    if (ctx->profiling) cudaEventRecord(ctx->pev[2 * pk], st);
    bool persistent_ran = false;
    if (key_multi) {
        e = launch_tiled<true>(ap, pl, 1, Lmax, st, maps);
        if (e == cudaSuccess) {
            ap.keyed_multi = 1;
        } else if (e == cudaErrorCooperativeLaunchTooLarge) {
            (void)cudaGetLastError();                        // the grid cannot be co-resident right now: one launch per layer does it all
        } else {
            return e;
        }
        ap.tile_done = nullptr;
    }
    if (persistent) {
        // packed kernel first where possible, then the 32-bit one: each returns at once unless it is the one chosen
        e = will_p16 ? launch_tiled<false>(ap, pl, 1, Lmax, st, maps, true) : cudaSuccess;
        if (e == cudaSuccess) e = launch_tiled<false>(ap, pl, 1, Lmax, st, maps);
        if (e == cudaErrorCooperativeLaunchTooLarge) {
            // the grid cannot be co-resident right now (SMs taken by another context): one launch per layer instead.
            // If the packed kernel was accepted before the 32-bit one was refused it may have run every layer, and on
            // the rolling buffer that overwrote layer 0: write the base layer again behind it.
            (void)cudaGetLastError();
            ap.tile_done = nullptr;
            if (!a.C && will_p16) {
                base_layer();
                if ((e = cudaGetLastError()) != cudaSuccess) return e;
            }
        } else if (e != cudaSuccess) {
            return e;
        } else {
            persistent_ran = true;
        }
    }
    for (int l = 1; l < Lmax && !persistent_ran; ++l) {
        if (reference) {
            const int mchunks = (a.m_pitch + 255) / 256;
            layer_reference_kernel<<<dim3((unsigned)((size_t)B * mchunks), S, 1), 256, 0, st>>>(a, l);
            e = cudaGetLastError();
        } else {
            e = a.A ? launch_tiled<true>(ap, pl, l, l + 1, st, maps) : launch_tiled<false>(ap, pl, l, l + 1, st, maps);
        }
        if (e != cudaSuccess) return e;
    }
    if (ctx->profiling) { cudaEventRecord(ctx->pev[2 * pk + 1], st); ++ctx->prof_count; }
    for (int b0 = 0; b0 < B; b0 += 65535) {                   // grid.y limit
        DpArgs c = a;
        const int nb = (B - b0 < 65535) ? B - b0 : 65535;
        c.L += b0; c.status += b0;
        if (c.C) c.C += (size_t)b0 * Lmax * S * a.m_pitch;
        c.C_last += (size_t)b0 * S * a.m_pitch;
        c.roll += (size_t)b0 * S * a.m_pitch;
        size_t per = ((size_t)S * a.m_pitch / 4 + 255) / 256;
        if (per > 64) per = 64;
        copy_last_kernel<<<dim3((unsigned)per, nb), 256, 0, st>>>(c);
    }
    finalize_kernel<<<(B + 255) / 256, 256, 0, st>>>(B, a.err, a.status);
    return cudaGetLastError();
}
