// Internal declarations shared by the translation units of libgalv.so.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

#include "galv.h"

struct galv_ctx {
    int device;
    int num_sms;
    int smem_optin;      // max dynamic shared memory per block (bytes)
    int max_cluster;     // largest thread-block cluster the cluster kernel may be launched with (8 portable, 16 where allowed)
    int profiling;       // record an event pair around the layer launches of every search
    int prof_count;      // searches profiled since profiling was switched on
    cudaEvent_t pev[2 * 64];   // ring of event pairs: search k uses pev[2*(k%64)], pev[2*(k%64)+1]
    char err[512];
};

// How one layer of the recurrence is cut into work items (host-chosen, passed to the kernels).
struct DpPlan {
    int tm;        // 32-column groups per warp (register tile height)
    int sb;        // strategies per item (s-block), multiple of 8
    int nsb;       // s-blocks
    int nsg;       // warps along s  (= sb / 8)
    int nms;       // warps along m
    int tmb;       // budget columns per item = nms * 32 * tm
    int ks;        // previous-layer strategies staged per pipeline stage
    int nkc;       // chunks per item = ceil(S / ks)
    int nst;       // pipeline stages in shared memory
    int tma_t;     // trans rows are 16-byte aligned: staged by a tiled TMA box, else by plain copies
    int ntiles_m;  // ceil((M+1) / tmb)
    int threads;   // (nsg * nms + 4) * 32: consumer warps, producer, helper, store and publisher warps
    int smem;      // dynamic shared memory bytes
    int grid;      // resident CTAs
    int p16;       // the packed 16-bit path is possible for this shape (whether the costs allow it is known on the device)
    int p16_smem;  // its dynamic shared memory bytes
};

struct DpArgs {
    int B, Lmax, S, M, m_pitch;
    const int32_t* L;
    const int32_t* time_q;
    const int32_t* mem_q;
    const int32_t* trans_q;
    long long trans_inst;   // entries per instance in trans_q: S*S, or Lmax*S*S with one matrix per layer
    long long trans_layer;  // entries between the matrices of consecutive layers: 0 or S*S
    int32_t* C;          // full table or NULL
    uint8_t* A;          // argmin table or NULL
    int32_t* C_last;
    int32_t* roll;       // [2][B][S][m_pitch] when C == NULL
    int32_t* order;      // [B]   valid instances, longest first
    int32_t* nactive;    // [Lmax+1] instances with L > l
    int32_t* scratch;    // [2*(Lmax+2)] histogram / fill counters, then the work counters below (zeroed together)
    unsigned long long* work;  // [Lmax+2] next item to hand out: [0] when all layers are one launch, else [l]
    long long* istart;   // [Lmax+1] items of the layers before l (layer 1 starts at 0); [Lmax] = all items
    int32_t* err;        // device error flag
    int32_t* tile_done;  // [B][ntiles_m] finished items per (instance, tile); NULL when layers are separate launches
    int32_t* maxmem;     // largest mem over the valid instances (min(.., M+1)); [1] largest trans entry; [2] 1: packed 16-bit path;
                         // [3] 1: trans_k holds shifted entries (keyed argmin loop)
    uint32_t* trans_p;   // packed pairs of trans rows for the 16-bit path: [B][(Lmax)][S/2][S], entry = T[2q][s] | T[2q+1][s] << 16
    int32_t* trans_k;    // argmin table with keys: copy of trans_q with every entry << 6 (same place in the workspace as trans_p;
                         // a plain copy when the entries are too large for keys: maxmem[3] says which)
    int keyed_multi;     // the keys-only argmin kernel has been launched over all layers: launches per layer return when it ran
    int keyed;           // the shape allows the keyed argmin loop (S <= 64, all rows of a tile in one stage)
    int32_t* minmem_l;   // [Lmax+1] smallest mem of each layer over the valid instances
    int32_t* front;      // [B][Lmax] feasibility frontier (sum of the layers' smallest mem), or NULL when tiles are never skipped
    int32_t* ntiles;     // [Lmax+1] tiles per instance that can store anything in layer l
    int32_t* tcount;     // [Lmax][ntiles_m] layers 1..l whose items include tile t
    int32_t* status;
    int withhold;        // test hook: CTA 0 never loads its first chunk, so that the bounded waits run out
    int skip_dom;        // packed path: leave out row pairs that cannot win in any column of a warp group's tile
};

// records `text` as the context's last error and returns `code`
int galv_set_error(galv_ctx* ctx, int code, const char* text);

// workspace carve-up (offsets in bytes, all 256-aligned)
struct WsLayout { size_t order, nactive, scratch, err, minmem_l, ntiles, istart, tcount, front, tile_done, trans_p, roll, total; };
WsLayout galv_ws_layout(const galv_shape* sh);

// How the cluster kernel (small batches: one thread-block cluster per instance) cuts an instance.
struct ClPlan {
    int cl;        // CTAs per cluster
    int w;         // budget columns per CTA (multiple of 32)
    int g;         // w / 32
    int nsg;       // ceil(S / 8)
    int sp8;       // nsg * 8
    int tm;        // 32-column groups per warp register tile
    int nct;       // column tiles per CTA
    int units;     // nct * nsg work units per CTA and layer
    int nw;        // warps per CTA
    int smem;      // dynamic shared memory bytes
    int sorted;    // clusters take the instances longest first
};
bool galv_cluster_plan(const galv_ctx* ctx, const galv_shape* sh, ClPlan* plan);
cudaError_t galv_cluster_configure(galv_ctx* ctx);
cudaError_t galv_cluster_launch(galv_ctx* ctx, const galv_shape* sh, const ClPlan& plan, const struct DpArgs& a, cudaStream_t st);

bool galv_dp_make_plan(const galv_ctx* ctx, const galv_shape* sh, DpPlan* plan);
cudaError_t galv_dp_configure(const galv_ctx* ctx);
cudaError_t galv_dp_launch(galv_ctx* ctx, const galv_shape* sh, const DpArgs& a, cudaStream_t st);
inline long long galv_trans_layer(const galv_shape* sh) { return (sh->flags & GALV_TRANS_PER_LAYER) ? (long long)sh->S * sh->S : 0; }
inline long long galv_trans_inst(const galv_shape* sh) { return (long long)sh->S * sh->S * ((sh->flags & GALV_TRANS_PER_LAYER) ? sh->Lmax : 1); }
cudaError_t galv_backtrack_launch(const galv_shape* sh, const int32_t* L, const int32_t* time_q,
                                  const int32_t* mem_q, const int32_t* trans_q, const int32_t* C,
                                  const uint8_t* A, const int32_t* C_last, const int32_t* budget,
                                  int32_t* opt_cost, int32_t* plan, int32_t* mem_used, int32_t* status,
                                  cudaStream_t st);
cudaError_t galv_costs_launch(const galv_shape* sh, const int32_t* L, const galv_layer_desc* layers,
                              int64_t layer_stride_B, const galv_strategy_desc* strat,
                              const galv_inst_params* inst, double* time_s, double* mem_bytes,
                              int32_t* time_q, int32_t* mem_q, int32_t* trans_q, int32_t* status,
                              cudaStream_t st);
cudaError_t galv_probe_launch(const galv_ctx* ctx, int kind, int iters, int32_t* sink, cudaStream_t st,
                              long long* ops);
