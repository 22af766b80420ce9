// Small batches: one thread-block cluster per search instance, the table slice kept in shared memory.
//
//   C[l][m][s] = time(l,s) + min_{s'} ( C[l-1][m-mem(l,s)][s'] + trans(s',s) )
//
// (Section 3 of the paper: the selector searches again while the job runs, one model at a time;
// Section 4: the manager's step.  Such a re-search is a batch of one to a few dozen instances.)
//
// With fewer work items per layer than the GPU has SMs the tiled kernel's step is a chain of dependent
// layers, each link paying a trip through L2 and a gpu-scope publish.  Here the chain never leaves the
// SMs: the budget columns of ONE instance are split over the CTAs of a cluster (CTA r owns columns
// r*W .. r*W+W-1), each CTA keeps its columns of the previous layer, all S rows, in shared memory,
// computes G[s][m'] = min_{s'}(Cprev[s'][m'] + T[s'][s]) for its own columns m' (no halo: G does not
// depend on mem) and PUSHES time + G to where it belongs, column m' + mem(l,s) of the next layer's
// buffer, which lies in its own shared memory or in that of a CTA further up: a plain store into
// distributed shared memory.  One hardware cluster barrier per layer (release / acquire) ends the
// layer.  Cells no column maps to (m < mem(l,s)) are written +inf by the CTA that owns them.
// The finished slice of a layer goes to the table in HBM by ONE tensor-map bulk store (TMA) straight
// from the shared-memory buffer, issued by a service warp while the other warps compute the next layer.
//
// The kernel validates its instance itself, writes the base layer, every layer and C_last: the
// whole search is one launch.  No spin-waits anywhere: the cluster barrier is a hardware barrier
// among co-scheduled CTAs, and clusters never wait on one another.  No cluster multicast.

#include <cuda.h>

#include <cstring>
#include <map>
#include <mutex>
#include <type_traits>

#include "galv_internal.h"


namespace {

constexpr int kInf = GALV_INF;
constexpr int kMaxSortedB = 512;          // instances whose lengths fit the ranking scratch below
constexpr int kRowsPerLane = 4;           // strategies per lane of the service warp: S <= 128

struct ClArgs {
    int B, Lmax, S, M, m_pitch;
    int CL;            // CTAs per cluster
    int W;             // budget columns per CTA (multiple of 32)
    int G;             // W / 32
    int NSG;           // ceil(S / 8)
    int SP8;           // NSG * 8: row pitch of the trans matrix in shared memory
    int nct;           // column tiles of 32*TM columns per CTA
    int units;         // nct * NSG work units per CTA and layer
    int sorted;        // clusters take the instances longest first
    const int32_t* L;
    const int32_t* time_q;
    const int32_t* mem_q;
    const int32_t* trans_q;
    long long trans_inst, trans_layer;
    int32_t* C;        // full table or NULL
    int32_t* C_last;
    int32_t* status;
    int32_t* path;     // [4] device flags of the search: error, -, -, kernel that ran
};

// 3-D view of a table for the tensor-map store: [rows of S strategies per (instance, layer)][m_pitch / 32][32].
// A CTA's slice [S][G][32] in shared memory is then one box.

__device__ __forceinline__ uint32_t smem_addr(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
// address of the same shared-memory location in the CTA of rank `rank` of this cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster(uint32_t addr, int v) {
    asm volatile("st.shared::cluster.s32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void cluster_barrier() {
    __syncwarp();                                              // the aligned forms want the whole warp together
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// One box [S][G][32] from shared memory to element coordinates (0, g0, row0) of the table behind `map`;
// what lies beyond the tensor's edge (the last CTA's columns past m_pitch) is not written.
__device__ __forceinline__ void tensor_store_3d(const CUtensorMap* map, const void* src, int g0, int row0) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];"
                 ::"l"(map), "r"(0), "r"(g0), "r"(row0), "r"(smem_addr(src)) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void cp_async_4(void* dst, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_addr(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// What the push of one (column tile, strategy) needs, derived once per layer and CTA by the service warp.
// Column m' of strategy s belongs at column m' + mem(l,s); for the tile that starts at this CTA's column colb:
//   x = CTA of the cluster that receives the tile's first column (-1: nothing of the tile lands inside the budget),
//   y = offset of that first column inside the receiving CTA's columns, z = time(l,s),
//   w = kWholeTile when all nj*32 columns land in CTA x, else the largest offset that still lands inside the
//       budget (the tile then straddles two CTAs or the budget's edge and every column is checked).
// mem is clamped to M+1: nothing it shifts by lands inside the budget.  Pad strategies (s >= S) get x = -1.
constexpr int kWholeTile = 0x7fffffff;
__device__ __forceinline__ int4 tile_record(bool real, int mem, int time, int M, int W, int rank, int colb, int ncols) {
    const int mc = mem < M + 1 ? mem : M + 1;
    const int q = mc / W;
    int d = rank + q, xb = colb + (mc - q * W);
    if (xb >= W) { xb -= W; ++d; }
    const int lim = M - d * W;
    if (!real || lim < xb) return make_int4(-1, 0, time, 0);
    const bool whole = xb + ncols <= W && xb + ncols - 1 <= lim;
    return make_int4(d, xb, time, whole ? kWholeTile : lim);
}
// cells of this CTA's own columns that no column maps to (m < mem): written +inf
__device__ __forceinline__ int fill_count(bool real, int mem, int M, int W, int rank) {
    const int mc = mem < M + 1 ? mem : M + 1;
    const int nf = mc - rank * W;
    return !real ? 0 : (nf < 0 ? 0 : (nf > W ? W : nf));
}

// One cluster per instance (cluster c takes the c-th longest when `sorted`), CTA `rank` of the cluster owns
// budget columns rank*W .. rank*W+W-1.  Dynamic shared memory: two buffers [S][W] of table values (previous
// and next layer, swapping), the transition matrix [S][SP8] (two of them with one matrix per layer), the push
// records of this layer and the next (one per column tile and strategy), the fill counts, and a dump row for the
// stores of strategies that land nowhere.  Warps 0..NW-1 compute: warp w takes work units w, w+NW, ...; a unit is
// 32*TM columns x 8 strategies, one fused add-min per relaxation, accumulators in registers.  The last warp
// is the service warp: it sends the finished layer to the table (one tensor-map store), prepares the next
// layer's records and, with one matrix per layer, fetches the next matrix.
template <int TM>
__global__ void __launch_bounds__(416, 1) cluster_search_kernel(const ClArgs a, const __grid_constant__ CUtensorMap map_c,
                                                                const __grid_constant__ CUtensorMap map_last)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ int s_L[kMaxSortedB];
    __shared__ int s_inst, s_tmax, s_bad;
    __shared__ long long s_sum;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, NT = blockDim.x, NW = (NT >> 5) - 1;
    const int CL = a.CL, rank = (int)cluster_rank(), cid = blockIdx.x / CL;
    const int S = a.S, M = a.M, W = a.W, SP8 = a.SP8, Lmax = a.Lmax;

    int32_t* const buf0 = reinterpret_cast<int32_t*>(smem_raw);
    int32_t* const buf1 = buf0 + S * W;
    int32_t* const tsm = buf1 + S * W;
    const int tmat = S * SP8;
    const int nrec = a.nct * SP8;
    int4* const rows = reinterpret_cast<int4*>(tsm + (a.trans_layer ? 2 : 1) * tmat);     // [2][nct][SP8] push records
    int* const fillc = reinterpret_cast<int*>(rows + 2 * nrec);                            // [2][SP8] leading cells of each row to fill with +inf
    int* const fillmax = fillc + 2 * SP8;                                                  // [2] the largest of them (padded to 4 ints)
    int32_t* const dump = fillmax + 4;                                                     // [32 * TM] where stores of skipped strategies go
    int* const cdelta = dump + 32 * TM;                                                    // [16] cluster-window address of CTA d minus this CTA's own shared address

    if (blockIdx.x == 0 && tid == 0) { a.path[0] = 0; a.path[3] = 2; }      // no error flag to raise; the cluster kernel ran

    // ---- which instance: clusters are dispatched in order, so the longest instances go first
    int i = cid;
    if (a.sorted) {
        for (int j = tid; j < a.B; j += NT) {
            const int v = a.L[j];
            s_L[j] = (v < 1 || v > Lmax) ? 0 : v;
        }
        __syncthreads();
        for (int j = tid; j < a.B; j += NT) {
            const int Lj = s_L[j];
            int before = 0;
            for (int k = 0; k < a.B; ++k) {
                const int Lk = s_L[k];
                before += (Lk > Lj) || (Lk == Lj && k < j);
            }
            if (before == cid) s_inst = j;
        }
        __syncthreads();
        i = s_inst;
    }

    // ---- validation (every CTA of the cluster comes to the same result: nobody is left waiting at a barrier)
    if (tid == 0) { s_sum = 0; s_tmax = 0; s_bad = 0; }
    __syncthreads();
    const int Li = a.L[i];
    if (Li < 1 || Li > Lmax) {
        if (rank == 0 && tid == 0) a.status[i] = GALV_STATUS_BAD_INPUT;
        return;
    }
    const int32_t* const tq = a.time_q + (size_t)i * Lmax * S;
    const int32_t* const mq = a.mem_q + (size_t)i * Lmax * S;
    const int32_t* const T0 = a.trans_q + (size_t)i * a.trans_inst;
    {
        long long sum = 0;
        int bad = 0, tmax = 0;
        for (int l = warp; l < Li; l += NW + 1) {             // a warp per layer: largest time of the layer
            int mx = 0;
            for (int s = lane; s < S; s += 32) {
                const int tv = tq[l * S + s], mv = mq[l * S + s];
                bad |= (tv < 0) | (mv < 0);
                mx = max(mx, tv);
            }
            mx = __reduce_max_sync(0xffffffffu, mx);
            if (lane == 0) sum += mx;
        }
        const int xl0 = a.trans_layer ? 1 : 0, xl1 = a.trans_layer ? Li : 1;       // matrices in use
        const long long nx = (long long)(xl1 - xl0) * S * S;
        const int32_t* x = T0 + (size_t)xl0 * S * S;
        for (long long k = tid; k < nx; k += NT) {
            const int v = x[k];
            bad |= (v < 0);
            tmax = max(tmax, v);
        }
        tmax = __reduce_max_sync(0xffffffffu, tmax);
        bad = __any_sync(0xffffffffu, bad != 0);
        if (lane == 0) {
            if (sum) atomicAdd(reinterpret_cast<unsigned long long*>(&s_sum), static_cast<unsigned long long>(sum));
            atomicMax(&s_tmax, tmax);
            if (bad) atomicOr(&s_bad, 1);
        }
    }
    __syncthreads();
    {
        int st = 0;
        if (s_bad) st = GALV_STATUS_BAD_INPUT;
        else if (s_sum + (long long)(Li - 1) * s_tmax >= (long long)kInf) st = GALV_STATUS_OVERFLOW_RISK;
        if (rank == 0 && tid == 0) a.status[i] = st;
        if (st) return;                                        // flagged: tables left untouched
    }

    const int col_g0 = rank * W;                               // first budget column of this CTA

    // ---- layer 0, the records of layer 1, the transition matrix
    // the push records and fill count of strategy s (raw mem / time given) into half `h` of the two arrays
    auto prepare_one = [&](int h, int s, int mem, int time) -> int {                       // returns the row's fill count
        const bool real = s < S;
        const int nf = fill_count(real, mem, M, W, rank);
        fillc[h * SP8 + s] = nf;
        for (int ct = 0; ct < a.nct; ++ct) {
            const int left = a.G - ct * TM;
            rows[h * nrec + ct * SP8 + s] = tile_record(real, mem, time, M, W, rank, ct * 32 * TM, 32 * (left < TM ? left : TM));
        }
        return nf;
    };
    // ... of a whole layer by one warp: lane k takes strategies k, k+32, ...
    auto prepare_layer = [&](int h, const int (&m)[kRowsPerLane], const int (&t)[kRowsPerLane]) {
        int most = 0;
#pragma unroll
        for (int j = 0; j < kRowsPerLane; ++j)
            if (lane + 32 * j < SP8) most = max(most, prepare_one(h, lane + 32 * j, m[j], t[j]));
        most = __reduce_max_sync(0xffffffffu, most);
        if (lane == 0) fillmax[h] = most;
    };
    // layers 0 and 1 straight from global memory, a warp each (nothing is being stored yet)
    if (warp <= 1 && warp < Li) {
        int m0[kRowsPerLane], t0[kRowsPerLane];
#pragma unroll
        for (int j = 0; j < kRowsPerLane; ++j) {
            const int s = lane + 32 * j;
            m0[j] = s < S ? mq[warp * S + s] : 0;
            t0[j] = s < S ? tq[warp * S + s] : 0;
        }
        prepare_layer(warp, m0, t0);
    }
    for (int x = tid; x < 32 * TM; x += NT) dump[x] = 0;
    // where the other CTAs' buffers lie in the cluster window: asked once, not once per store (the mapping is an
    // offset per CTA; asking inside the push puts its latency on every strategy's chain of branches)
    if (tid < 16) cdelta[tid] = (int)(map_to_rank(smem_addr(buf0), (uint32_t)min(tid, CL - 1)) - smem_addr(buf0));
    {
        const int32_t* T = T0 + (a.trans_layer ? a.trans_layer : 0);       // matrix 1 is paid between layers 0 and 1
        int32_t* dst = tsm + (a.trans_layer ? tmat : 0);                    // per layer: matrix l sits in tsm[l & 1]
        for (int e = tid; e < tmat; e += NT) {
            const int k = e / SP8, c = e - k * SP8;
            dst[e] = (c < S && Li > 1) ? T[k * S + c] : 0;
            if (a.trans_layer) tsm[e] = 0;                                  // pad columns of the other buffer stay 0
        }
    }
    __syncthreads();
    for (int s = warp; s < S; s += NW + 1) {
        const int t0 = rows[s].z;                                           // time(0,s) sits in every record of s
        const int nf = fillc[s];
        for (int x = lane; x < W; x += 32) {
            const bool pad = col_g0 + x > M;
            buf0[s * W + x] = (pad || x < nf) ? kInf : t0;
            if (pad) buf1[s * W + x] = kInf;                                // pad columns are never written again
        }
    }
    // Service warp: raw mem / time rows of the layer after next, lane k keeps strategies k, k+32, ... (S <= 128).
    // They are fetched a whole layer before they are needed and BEFORE that layer's table store is issued: a
    // global load issued while the SM's bulk stores are in flight comes back after thousands of cycles.
    int raw_m[kRowsPerLane], raw_t[kRowsPerLane];
    auto fetch_rows = [&](int lay, int (&m)[kRowsPerLane], int (&t)[kRowsPerLane]) {
#pragma unroll
        for (int j = 0; j < kRowsPerLane; ++j) {
            const int s = lane + 32 * j;
            m[j] = s < S ? mq[lay * S + s] : 0;
            t[j] = s < S ? tq[lay * S + s] : 0;
        }
    };
    if (warp == NW && Li > 2) fetch_rows(2, raw_m, raw_t);
    // every CTA of the cluster has started and holds its layer 0 before anyone writes into a neighbour
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");            // layer 0 goes to the table by a bulk store
    cluster_barrier();

    for (int l = 1; l < Li; ++l) {
        const int32_t* const X = (l & 1) ? buf0 : buf1;                     // layer l-1
        int32_t* const Y = (l & 1) ? buf1 : buf0;                           // layer l
        const int4* const rl = rows + (l & 1) * nrec;
        const int32_t* const Tl = tsm + ((a.trans_layer && (l & 1)) ? tmat : 0);

        if (warp == NW) {
            // ------------------------------------------------------------ service warp
            // first the loads: rows of layer l+2, and with one matrix per layer the matrix of layer l+1
            int next_m[kRowsPerLane], next_t[kRowsPerLane];
            if (l + 2 < Li) fetch_rows(l + 2, next_m, next_t);
            if (l + 1 < Li && a.trans_layer) {
                const int32_t* T = T0 + (size_t)(l + 1) * a.trans_layer;
                int32_t* dst = tsm + (((l + 1) & 1) ? tmat : 0);
                for (int e = lane; e < S * S; e += 32) {
                    const int k = e / S, c = e - k * S;
                    cp_async_4(dst + k * SP8 + c, T + e);
                }
            }
            // layer l-1 is complete in X: to the table while this layer is computed
            if (a.C && lane == 0) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");    // the buffer was written by plain stores
                tensor_store_3d(&map_c, X, rank * a.G, (i * Lmax + (l - 1)) * S);
                bulk_commit();
            }
            // the records of layer l+1 from the rows fetched a layer ago
            if (l + 1 < Li) prepare_layer((l + 1) & 1, raw_m, raw_t);
#pragma unroll
            for (int j = 0; j < kRowsPerLane; ++j) { raw_m[j] = next_m[j]; raw_t[j] = next_t[j]; }
            if (l + 1 < Li && a.trans_layer) cp_async_wait_all();
            if (a.C && lane == 0) bulk_wait_read();                         // X may be overwritten from the next barrier on
        } else {
            // ------------------------------------------------------------ compute warps
            // cells of this CTA's columns that no column maps to in this layer (m < mem(l,s): the first fillc[s] of
            // row s): the compute warps share the columns, each takes every strategy in turn (independent predicated
            // stores; a loop per strategy would be a chain of dependent steps)
            {
                const int* const fc = fillc + (l & 1) * SP8;
                const int most = fillmax[l & 1];
                for (int x = warp * 32 + lane; x < most; x += NW * 32) {
#pragma unroll 4
                    for (int s = 0; s < S; ++s)
                        if (x < fc[s]) Y[s * W + x] = kInf;
                }
            }
            const uint32_t ybase = smem_addr(Y);
            for (int unit = warp; unit < a.units; unit += NW) {
                const int ct = unit / a.NSG, sg = unit - ct * a.NSG;
                const int colb = ct * (32 * TM);
                int nj = a.G - ct * TM;                                     // 32-column groups of this tile that exist
                nj = nj > TM ? TM : nj;
                int acc[TM][8];
#pragma unroll
                for (int j = 0; j < TM; ++j)
#pragma unroll
                    for (int u = 0; u < 8; ++u) acc[j][u] = kInf;
                const int32_t* pc = X + colb + lane;
                const int32_t* pt = Tl + sg * 8;
                int k = 0;
                auto steps = [&](auto ku) {
                    constexpr int K = decltype(ku)::value;
                    for (; k + K <= S; k += K) {
#pragma unroll
                        for (int kk = 0; kk < K; ++kk) {
                            int c[TM];
#pragma unroll
                            for (int j = 0; j < TM; ++j) c[j] = pc[kk * W + j * 32];
                            const int4 t0 = *reinterpret_cast<const int4*>(pt + kk * SP8);
                            const int4 t1 = *reinterpret_cast<const int4*>(pt + kk * SP8 + 4);
                            const int t[8] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w};
#pragma unroll
                            for (int j = 0; j < TM; ++j)
#pragma unroll
                                for (int u = 0; u < 8; ++u) acc[j][u] = __viaddmin_s32(c[j], t[u], acc[j][u]);
                        }
                        pc += K * W;
                        pt += K * SP8;
                    }
                };
                steps(std::integral_constant<int, 8>());
                steps(std::integral_constant<int, 1>());
                // push: column m' of strategy s belongs at column m' + mem(l,s): in this CTA's buffer or in one further up.
                // All eight records first; when every strategy either stays at home in one piece or lands nowhere, the
                // stores go out in one run without a branch (those that land nowhere go to a dump row).
                int4 r[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) r[u] = rl[ct * SP8 + sg * 8 + u];
                bool plain = nj == TM;
#pragma unroll
                for (int u = 0; u < 8; ++u) plain = plain && (r[u].x < 0 || (r[u].x == rank && r[u].w == kWholeTile));
                int32_t* const yl = Y + (sg * 8) * W + lane;
                if (plain) {
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        int32_t* const y = r[u].x < 0 ? dump + lane : yl + u * W + r[u].y;
#pragma unroll
                        for (int j = 0; j < TM; ++j) y[j * 32] = __viaddmin_s32(acc[j][u], r[u].z, kInf);    // +inf stays +inf
                    }
                } else {
                    // Some strategy's tile leaves the CTA or straddles two: the whole unit goes through the cluster window
                    // (what stays at home too), one predicated store a register and no branch - a chain of branches per
                    // strategy cost the warps that own such tiles three times the time of the stores themselves.
                    // A whole tile has w = the largest int: its columns pass the test against w and lie below W.
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const int dx = r[u].x < 0 ? 0 : r[u].x;
                        const uint32_t row = ybase + (uint32_t)((sg * 8 + u) * W) * 4u;
                        const uint32_t ra0 = row + (uint32_t)cdelta[dx];
                        const uint32_t ra1 = row + (uint32_t)cdelta[min(dx + 1, CL - 1)] - (uint32_t)W * 4u;
                        const bool lands = r[u].x >= 0;
#pragma unroll
                        for (int j = 0; j < TM; ++j)
                            if (j < nj) {
                                const int x = r[u].y + j * 32 + lane;
                                const int v = __viaddmin_s32(acc[j][u], r[u].z, kInf);
                                if (lands && x <= r[u].w) st_cluster((x < W ? ra0 : ra1) + (uint32_t)x * 4u, v);
                            }
                    }
                }
            }
        }
        // What this thread stored into shared memory, its own CTA's or a neighbour's, is read next by the bulk store of
        // the CTA that owns it (async proxy): the writer orders it for that proxy before the barrier that publishes it.
        asm volatile("fence.proxy.async.shared::cluster;" ::: "memory");
        cluster_barrier();                                                  // layer l is complete everywhere
    }

    // ---- the last layer: to the table and to C_last
    if (warp == NW && lane == 0) {
        const int32_t* const F = ((Li - 1) & 1) ? buf1 : buf0;
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        if (a.C) tensor_store_3d(&map_c, F, rank * a.G, (i * Lmax + (Li - 1)) * S);
        tensor_store_3d(&map_last, F, rank * a.G, i * S);
        bulk_commit();
        bulk_wait_all();
    }
}

}  // namespace

// ---------------------------------------------------------------- host side

namespace {

typedef CUresult (*PFN_encodeTiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                    const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Tensor map of an int32 table [rows][m_pitch] seen as [rows][m_pitch / 32][32], box [box_rows][box_groups][32].
cudaError_t encode_table_3d(CUtensorMap* map, void* base, size_t rows, int m_pitch, int box_rows, int box_groups)
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
    const cuuint64_t dims[3] = {32, (cuuint64_t)(m_pitch / 32), (cuuint64_t)rows};
    const cuuint64_t strides[2] = {128, (cuuint64_t)m_pitch * 4};
    const cuuint32_t box[3] = {32, (cuuint32_t)box_groups, (cuuint32_t)box_rows};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_INT32, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

template <int TM>
cudaError_t launch_cluster(const ClArgs& a, const ClPlan& p, const CUtensorMap& mc, const CUtensorMap& ml, cudaStream_t st, int* max_clusters)
{
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)(a.B * p.cl));
    cfg.blockDim = dim3((unsigned)((p.nw + 1) * 32));
    cfg.dynamicSmemBytes = (size_t)p.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)p.cl;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (max_clusters) return cudaOccupancyMaxActiveClusters(max_clusters, cluster_search_kernel<TM>, &cfg);
    return cudaLaunchKernelEx(&cfg, cluster_search_kernel<TM>, a, mc, ml);
}

cudaError_t launch_any(const ClArgs& a, const ClPlan& p, const CUtensorMap& mc, const CUtensorMap& ml, cudaStream_t st, int* max_clusters)
{
    switch (p.tm) {
    case 2: return launch_cluster<2>(a, p, mc, ml, st, max_clusters);
    case 3: return launch_cluster<3>(a, p, mc, ml, st, max_clusters);
    default: return launch_cluster<4>(a, p, mc, ml, st, max_clusters);
    }
}

// Clusters of this plan's size and resources the device can hold at once (asked once per kind of launch).
int max_active_clusters(const galv_ctx* ctx, const ClPlan& p)
{
    static std::map<unsigned long long, int> cache;          // shared by all contexts of the process
    static std::mutex cache_mutex;
    std::lock_guard<std::mutex> lock(cache_mutex);
    const unsigned long long key = ((unsigned long long)ctx->device << 48) | ((unsigned long long)p.cl << 40) |
                                   ((unsigned long long)p.tm << 36) | ((unsigned long long)p.nw << 28) | (unsigned long long)((p.smem + 1023) / 1024);
    auto it = cache.find(key);
    if (it != cache.end()) return it->second;
    ClArgs a{};
    a.B = 1;
    CUtensorMap m{};
    int n = 0;
    if (launch_any(a, p, m, m, nullptr, &n) != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
    cache[key] = n;
    return n;
}

// Register-tile height for g column groups per CTA: the one that gives the busiest warp the least work (units are
// dealt out to at most 12 warps), then the busiest scheduler, then the smaller tile (more, smaller units spread the
// cost of the tiles that straddle two CTAs).  Returns the busiest scheduler's work in units of 8*S*2 cycles.
int tile_cost(int g, int nsg, int* tm_out)
{
    int best_tm = 4, best_warp = 1 << 30, best_sched = 1 << 30;
    for (int tm = 4; tm >= 2; --tm) {
        const int units = (g + tm - 1) / tm * nsg;
        int nw = (units + 3) & ~3;
        if (nw > 12) nw = 12;
        const int warp = (units + nw - 1) / nw * tm;
        const int sched = (units + 3) / 4 * tm;
        if (warp < best_warp || (warp == best_warp && sched <= best_sched)) { best_warp = warp; best_sched = sched; best_tm = tm; }
    }
    *tm_out = best_tm;
    return best_sched;
}

}  // namespace

// Whether the cluster kernel can run this shape, and how: CTAs per cluster, columns per CTA, register tile.
bool galv_cluster_plan(const galv_ctx* ctx, const galv_shape* sh, ClPlan* out)
{
    std::memset(out, 0, sizeof(*out));
    if (sh->flags & (GALV_STORE_ARGMIN | GALV_KERNEL_REFERENCE | GALV_KERNEL_PER_LAYER | GALV_DEBUG_WITHHOLD_LOAD | GALV_KERNEL_NO_CLUSTER))
        return false;
    const int S = sh->S, Gt = sh->m_pitch / 32;
    if (S > 32 * kRowsPerLane) return false;
    if ((long long)sh->B * sh->Lmax * S >= (1ll << 31)) return false;       // row coordinates of the table store are 32-bit
    const int nsg = (S + 7) / 8, sp8 = nsg * 8;
    const int nT = (sh->flags & GALV_TRANS_PER_LAYER) ? 2 : 1;
    const int budget = ctx->smem_optin - 4096;               // static shared memory of the kernel, rounded up
    // Candidates: every cluster size that gives each CTA at least 96 columns and leaves none without columns.
    // Estimated SM cycles per layer of a cluster, fitted to measurements on B200: the add-min issue time of the
    // busiest scheduler, stretched by the per-cell work beside it (push, fill, shared-memory loads: about 24
    // add-mins' worth per cell), plus what a layer costs whatever its size (barrier, drain of the pushes that
    // cross CTAs, start): about 3000 cycles, some more for clusters beyond 12 CTAs.  With more instances than the
    // device holds clusters the batch takes several rounds; on its own the kernel is chosen only when one round
    // does (a batch that needs rounds is better off on the tiled kernels, whose SMs never wait on a barrier).
    double best_time = 0.0;
    bool found = false;
    const int want_cl = (sh->flags >> 16) & 31;              // GALV_CLUSTER_SIZE(n): only clusters of n CTAs
    const bool forced = (sh->flags & GALV_KERNEL_CLUSTER) != 0 || want_cl != 0;
    for (int cl = ctx->max_cluster; cl >= 1; --cl) {
        if (want_cl && cl != want_cl) continue;
        const int g = (Gt + cl - 1) / cl;
        if (cl > 1 && (g < 3 || g * (cl - 1) >= Gt)) continue;
        const long long smem = (long long)2 * S * g * 32 * 4 + (long long)nT * S * sp8 * 4 + (long long)2 * ((g + 1) / 2) * sp8 * 16 + (long long)2 * sp8 * 4 + 16 + 512 + 64;
        if (smem > budget) break;                            // smaller clusters need more per CTA
        ClPlan p;
        std::memset(&p, 0, sizeof(p));
        p.cl = cl; p.g = g; p.w = g * 32; p.nsg = nsg; p.sp8 = sp8;
        const int cost = tile_cost(g, nsg, &p.tm);
        p.nct = (g + p.tm - 1) / p.tm;
        p.units = p.nct * nsg;
        p.nw = (p.units + 3) & ~3;                           // a multiple of 4: the SM's four schedulers get the same share
        if (p.nw > 12) p.nw = 12;
        p.smem = (int)smem;
        const int slots = max_active_clusters(ctx, p);
        if (slots < 1) continue;
        if (!forced && sh->B > slots) continue;
        const double rounds = (double)((sh->B + slots - 1) / slots);
        const double active = (double)(sh->B < slots ? sh->B : slots) * cl;     // CTAs resident at once
        const double share = active > ctx->num_sms ? active / ctx->num_sms : 1.0;   // ... of which this many share an SM's ALUs
        const double t = rounds * ((double)cost * 16.0 * S * (1.0 + 24.0 / S) * share + 3000.0 + (cl > 12 ? 800.0 : 0.0));
        if (!found || t < best_time) {
            best_time = t;
            found = true;
            p.sorted = sh->B > slots;                        // more clusters than fit at once: the longest instances first
            *out = p;
        }
    }
    if (!found) return false;
    if (out->sorted && sh->B > kMaxSortedB) return false;
    return true;
}

cudaError_t galv_cluster_configure(galv_ctx* ctx)
{
    const int bytes = ctx->smem_optin - 4096;
    cudaError_t e = cudaFuncSetAttribute(cluster_search_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(cluster_search_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(cluster_search_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) return e;
    // clusters of up to 16 CTAs where the device allows them (beyond the portable 8)
    ctx->max_cluster = 8;
    if (cudaFuncSetAttribute(cluster_search_kernel<2>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess &&
        cudaFuncSetAttribute(cluster_search_kernel<3>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess &&
        cudaFuncSetAttribute(cluster_search_kernel<4>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess)
        ctx->max_cluster = 16;
    else
        (void)cudaGetLastError();
    return cudaSuccess;
}

cudaError_t galv_cluster_launch(galv_ctx* ctx, const galv_shape* sh, const ClPlan& p, const DpArgs& d, cudaStream_t st)
{
    ClArgs a;
    a.B = d.B; a.Lmax = d.Lmax; a.S = d.S; a.M = d.M; a.m_pitch = d.m_pitch;
    a.CL = p.cl; a.W = p.w; a.G = p.g; a.NSG = p.nsg; a.SP8 = p.sp8; a.nct = p.nct; a.units = p.units; a.sorted = p.sorted;
    a.L = d.L; a.time_q = d.time_q; a.mem_q = d.mem_q; a.trans_q = d.trans_q;
    a.trans_inst = d.trans_inst; a.trans_layer = d.trans_layer;
    a.C = d.C; a.C_last = d.C_last; a.status = d.status; a.path = d.err;
    (void)sh;
    CUtensorMap mc, ml;
    std::memset(&mc, 0, sizeof(mc));
    cudaError_t e = encode_table_3d(&ml, d.C_last, (size_t)d.B * d.S, d.m_pitch, d.S, p.g);
    if (e == cudaSuccess && d.C) e = encode_table_3d(&mc, d.C, (size_t)d.B * d.Lmax * d.S, d.m_pitch, d.S, p.g);
    if (e != cudaSuccess) return e;
    const int pk = ctx->prof_count % 64;
    if (ctx->profiling) cudaEventRecord(ctx->pev[2 * pk], st);
    e = launch_any(a, p, mc, ml, st, nullptr);
    if (e != cudaSuccess) return e;
    if (ctx->profiling) { cudaEventRecord(ctx->pev[2 * pk + 1], st); ++ctx->prof_count; }
    return cudaGetLastError();
}
