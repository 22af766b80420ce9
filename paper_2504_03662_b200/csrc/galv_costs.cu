// Cost model of the strategy search: fp64, elementwise.
//
// (Section 3 of the paper: the selector builds a performance model from the
// model profiler's per-layer shapes and FLOPs, the hardware profiler's memory
// and link bandwidth, and the dataset profiler's batch.)
//
// This translation unit is compiled with -fmad=false: every product and sum is
// rounded on its own, in the order written, so the doubles equal what any IEEE
// host computes from the same expression tree.
//
// The element (instance i, layer l, strategy s) depends on l only through the
// layer's descriptor, and a transformer stack repeats a handful of layer kinds
// (one in a uniform decoder, two in an attention / FFN stack).  So one CTA per
// instance first finds, for every layer, the nearest earlier layer (within a
// small window) with the very same descriptor bytes, evaluates the expression
// once per distinct layer and strategy into shared memory, and then writes the
// rows of all layers from there with 128-bit stores: the fp64 work (some
// sixteen divisions per element, each rounded on its own) shrinks by the
// repeat factor and the pass becomes the write of its outputs.  Nothing is
// re-associated: a repeated layer gets the bits its first occurrence got,
// which are the bits the expression gives for it.
// The transition entries depend on the two strategies only through their
// tensor-parallel degree, sequence-parallel flag and batch divisor: they are
// evaluated once per pair of such classes and written out from a small table.

#include "galv_internal.h"

namespace {

constexpr int kWindow = 8;         // how far back a layer looks for its twin
constexpr int kThreads = 256;

__device__ __forceinline__ int32_t quant_time(double t_s, double unit_ns) {
    double q = rint(t_s * 1e9 / unit_ns);
    if (!(q < 1073741824.0)) q = 1073741824.0;
    if (q < 0.0) q = 0.0;
    return (int32_t)q;
}

__device__ __forceinline__ int32_t quant_mem(double bytes, double bin_bytes) {
    double q = ceil(bytes / bin_bytes);
    if (!(q < 1073741824.0)) q = 1073741824.0;
    if (q < 0.0) q = 0.0;
    return (int32_t)q;
}

__device__ __forceinline__ bool pos_finite(double x) { return x > 0.0 && x < INFINITY; }
__device__ __forceinline__ bool nonneg_finite(double x) { return x >= 0.0 && x < INFINITY; }

// Descriptors no profiler could have produced: a rate, size or divisor that is not a positive finite number, a
// degree below 1, a ZeRO stage outside 0..3, a flag that is not 0/1, a negative coefficient.
__device__ __forceinline__ bool inst_ok(const galv_inst_params& in) {
    return pos_finite(in.b) && pos_finite(in.act_mult) && pos_finite(in.flops_rate) && pos_finite(in.bw_tp) && pos_finite(in.bw_dp) &&
           pos_finite(in.bytes_per_elem) && pos_finite(in.bin_bytes) && pos_finite(in.time_unit_ns);
}
__device__ __forceinline__ bool strat_ok(const galv_strategy_desc& sd) {
    return sd.tp >= 1 && sd.dp >= 1 && sd.zero >= 0 && sd.zero <= 3 && (sd.ckpt == 0 || sd.ckpt == 1) && (sd.sp == 0 || sd.sp == 1) &&
           pos_finite(sd.batch_div);
}
__device__ __forceinline__ bool layer_ok(const galv_layer_desc& ly) {
    return pos_finite(ly.h) && pos_finite(ly.seq) && nonneg_finite(ly.heads) && nonneg_finite(ly.c_lin) && nonneg_finite(ly.c_attn) &&
           nonneg_finite(ly.p_coef) && nonneg_finite(ly.n_ar) && nonneg_finite(ly.act_rep) && nonneg_finite(ly.act_tp) &&
           nonneg_finite(ly.act_attn);
}

// time_s and mem_bytes of one (layer, strategy, instance): the expression tree of the cost model, in this order.
__device__ __forceinline__ void cost_of(const galv_layer_desc& ly, const galv_strategy_desc& sd, const galv_inst_params& in,
                                        double* time_s, double* mem_bytes)
{
    const double tp = (double)sd.tp, dp = (double)sd.dp;
    const double bq = in.b / sd.batch_div;
    const double sbh = ly.seq * bq * ly.h;
    const double fwd = ly.c_lin * bq * ly.seq * ly.h * ly.h + ly.c_attn * bq * ly.seq * ly.seq * ly.h;
    const double t_comp = fwd * (3.0 + (double)sd.ckpt) / tp / in.flops_rate;
    const double t_tp = ly.n_ar * (2.0 * (tp - 1.0) / tp) * (bq * ly.seq * ly.h * in.bytes_per_elem) / in.bw_tp;
    const double zmul = sd.zero == 3 ? 1.5 : 1.0;
    const double t_dp = zmul * (2.0 * (dp - 1.0) / dp) * (ly.p_coef * ly.h * ly.h * in.bytes_per_elem / tp) / in.bw_dp;
    *time_s = (t_comp + t_tp) + t_dp;

    const double psi = ly.p_coef * ly.h * ly.h / tp;
    double zb;
    if (sd.zero == 0) zb = 16.0;
    else if (sd.zero == 1) zb = 4.0 + 12.0 / dp;
    else if (sd.zero == 2) zb = 2.0 + 14.0 / dp;
    else zb = 16.0 / dp;
    const double state = psi * zb;
    double act;
    if (sd.ckpt)
        act = sd.sp ? 2.0 * sbh / tp : 2.0 * sbh;
    else if (sd.sp)
        act = sbh * (ly.act_rep + ly.act_tp) / tp + ly.act_attn * ly.heads * ly.seq * ly.seq * bq / tp;
    else
        act = sbh * (ly.act_rep + ly.act_tp / tp) + ly.act_attn * ly.heads * ly.seq * ly.seq * bq / tp;
    *mem_bytes = state + in.act_mult * act;
}

__device__ __forceinline__ bool same_bytes(const galv_layer_desc* a, const galv_layer_desc* b) {
    const unsigned long long* x = reinterpret_cast<const unsigned long long*>(a);
    const unsigned long long* y = reinterpret_cast<const unsigned long long*>(b);
    bool eq = true;
#pragma unroll
    for (int k = 0; k < 10; ++k) eq = eq && x[k] == y[k];
    return eq;
}

// One CTA per instance.  Dynamic shared memory: root[Lmax] (the layer whose values layer l takes), slot[Lmax]
// (position of a distinct layer in the list), list[Lmax] (the distinct layers), then the table of one chunk of
// distinct layers: tq/mq int32 [KC][S] and, when the doubles are asked for, time_s/mem_bytes [KC][S].
__device__ __forceinline__ void cost_body(const int i, unsigned char* smem_raw, int Lmax, int S, int KC, const int32_t* __restrict__ L,
                                          const galv_layer_desc* __restrict__ layers, long long layer_stride_B,
                                          const galv_strategy_desc* __restrict__ strat,
                                          const galv_inst_params* __restrict__ inst, double* __restrict__ time_s,
                                          double* __restrict__ mem_bytes, int32_t* __restrict__ time_q,
                                          int32_t* __restrict__ mem_q, int32_t* __restrict__ trans_q,
                                          int32_t* __restrict__ status)
{
    __shared__ int s_bad, s_ndist;
    const int tid = threadIdx.x;
    const int Li = L[i];
    if (Li < 1 || Li > Lmax) {
        if (tid == 0) status[i] = GALV_STATUS_BAD_INPUT;       // nothing is written for this instance
        return;
    }
    int* const root = reinterpret_cast<int*>(smem_raw);
    int* const slot = root + Lmax;
    int* const list = slot + Lmax;
    int32_t* const tabq = list + Lmax + ((-3 * Lmax) & 3);      // 16-byte aligned: rows are read as int4
    int32_t* const tabm = tabq + KC * S;
    double* const tabt = reinterpret_cast<double*>(tabm + KC * S + ((2 * KC * S) & 1));
    double* const tabb = tabt + KC * S;
    const bool want_d = time_s != nullptr || mem_bytes != nullptr;

    const galv_layer_desc* const ly = layers + (long long)i * layer_stride_B;
    const galv_inst_params in = inst[i];
    if (tid == 0) { s_bad = inst_ok(in) ? 0 : 1; s_ndist = 0; }
    __syncthreads();
    // descriptors, and for every layer the nearest earlier twin
    bool bad = false;
    for (int s = tid; s < S; s += kThreads) bad = bad || !strat_ok(strat[s]);
    for (int l = tid; l < Li; l += kThreads) {
        bad = bad || !layer_ok(ly[l]);
        int parent = l;
        for (int d = 1; d <= kWindow && d <= l; ++d)
            if (same_bytes(ly + l, ly + l - d)) { parent = l - d; break; }
        root[l] = parent;
    }
    if (bad) atomicOr(&s_bad, 1);
    __syncthreads();
    const size_t base = (size_t)i * Lmax * S;
    if (s_bad) {
        // the whole instance is flagged; its integer tables say so to the search's validation as well
        if (tid == 0) status[i] = GALV_STATUS_BAD_INPUT;
        for (int e = tid; e < Li * S; e += kThreads) { time_q[base + e] = -1; mem_q[base + e] = -1; }
        for (int e = tid; e < S * S; e += kThreads) trans_q[(size_t)i * S * S + e] = -1;
        return;
    }
    if (tid == 0) status[i] = 0;
    // follow the twins back to the first of their kind by pointer jumping (a chain of twins can be as long as the
    // stack); the firsts form the list of distinct layers
    for (int l = tid; l < Li; l += kThreads)
        if (root[l] == l) { const int p = atomicAdd(&s_ndist, 1); list[p] = l; slot[l] = p; }
    for (int span = 1; span < Li; span <<= 1) {                // after k rounds every pointer has skipped 2^k twins or is home
        __syncthreads();
        volatile int* const vr = root;                         // a read may see this round's value or the last one: both are ancestors
        for (int l = tid; l < Li; l += kThreads) vr[l] = vr[vr[l]];
    }
    __syncthreads();
    for (int l = tid; l < Li; l += kThreads) root[l] = slot[root[l]];       // from here on: the position of layer l's kind in the list
    __syncthreads();
    const int ndist = s_ndist;
    const bool vec = (S & 3) == 0;
    for (int k0 = 0; k0 < ndist; k0 += KC) {
        const int kn = min(KC, ndist - k0);
        // the expression, once per distinct layer of this chunk and strategy
        for (int e = tid; e < kn * S; e += kThreads) {
            const int k = e / S, s = e - k * S;
            double t, b;
            cost_of(ly[list[k0 + k]], strat[s], in, &t, &b);
            tabq[e] = quant_time(t, in.time_unit_ns);
            tabm[e] = quant_mem(b, in.bin_bytes);
            if (want_d) { tabt[e] = t; tabb[e] = b; }
        }
        __syncthreads();
        // every layer whose kind is in this chunk takes its row from the table
        if (vec && (S >> 2) <= kThreads) {
            // a thread keeps its 16-byte column of the rows and walks down the layers: no division in the loop
            const int S4 = S >> 2, rows_per_pass = kThreads / S4;
            const int c = tid % S4, r0 = tid / S4;
            if (r0 < rows_per_pass)
                for (int l = r0; l < Li; l += rows_per_pass) {
                    const int k = root[l] - k0;
                    if (k < 0 || k >= kn) continue;
                    reinterpret_cast<int4*>(time_q + base + (size_t)l * S)[c] = reinterpret_cast<const int4*>(tabq + k * S)[c];
                    reinterpret_cast<int4*>(mem_q + base + (size_t)l * S)[c] = reinterpret_cast<const int4*>(tabm + k * S)[c];
                }
        } else {
            for (int e = tid; e < Li * S; e += kThreads) {
                const int l = e / S, s = e - l * S;
                const int k = root[l] - k0;
                if (k < 0 || k >= kn) continue;
                time_q[base + e] = tabq[k * S + s];
                mem_q[base + e] = tabm[k * S + s];
            }
        }
        if (want_d)
            for (int e = tid; e < Li * S; e += kThreads) {
                const int l = e / S, s = e - l * S;
                const int k = root[l] - k0;
                if (k < 0 || k >= kn) continue;
                if (time_s) time_s[base + e] = tabt[k * S + s];
                if (mem_bytes) mem_bytes[base + e] = tabb[k * S + s];
            }
        __syncthreads();
    }
}

// trans_q[i][a][c]: resharding time from strategy a (previous layer) to c (this layer):
//   ((k-1)/k + [sp changes] (tp_c-1)/tp_c) * (b/batch_div_c * seq * h * bytes_per_elem) / bw_tp,  k = ratio of the tp degrees.
// It depends on a through (tp, sp) and on c through (tp, sp, batch_div) only; strategies that agree in those form a
// class (8 classes among the 64 strategies of the heterogeneous workload).  A CTA finds the classes once, then for
// each of its instances evaluates the expression once per pair of classes and writes all S*S entries from that
// table: the same bits as evaluating every entry, at a fraction of the divisions.
__device__ __forceinline__ double pair_factor(const galv_strategy_desc& sa, const galv_strategy_desc& sc) {
    const double tpa = (double)sa.tp, tpc = (double)sc.tp;
    const double k = (tpa > tpc ? tpa : tpc) / (tpa < tpc ? tpa : tpc);
    const double spterm = (sa.sp != sc.sp) ? (tpc - 1.0) / tpc : 0.0;
    return (k - 1.0) / k + spterm;
}
// Dynamic shared memory: slot[S] (class of each strategy), rep[S] (one strategy per class), tab[ncls * ncls].
// status == nullptr: no earlier kernel has checked the descriptors; the CTA applies the cost kernel's own tests and
// leaves a flagged instance to it (which writes -1 everywhere).
__device__ __forceinline__ void trans_body(const int cta, unsigned char* smem_raw, int B, int Lmax, int S, const int32_t* __restrict__ L,
                                           const galv_layer_desc* __restrict__ layers, long long layer_stride_B,
                                           const galv_strategy_desc* __restrict__ strat,
                                           const galv_inst_params* __restrict__ inst, const int32_t* __restrict__ status,
                                           int32_t* __restrict__ trans_q, int inst_per_cta)
{
    __shared__ int s_ncls, s_sbad;
    int* const slot = reinterpret_cast<int*>(smem_raw);
    int* const rep = slot + S;
    int32_t* const tab = rep + S;
    const int tid = threadIdx.x;
    if (tid == 0) { s_ncls = 0; s_sbad = 0; }
    __syncthreads();
    // a strategy opens a class when no earlier one agrees with it in tp, sp and batch_div (compared as bits)
    for (int s = tid; s < S; s += kThreads) {
        const galv_strategy_desc me = strat[s];
        if (!status && !strat_ok(me)) atomicOr(&s_sbad, 1);
        int first = s;
        for (int o = 0; o < s; ++o) {
            const galv_strategy_desc ot = strat[o];
            if (ot.tp == me.tp && ot.sp == me.sp && __double_as_longlong(ot.batch_div) == __double_as_longlong(me.batch_div)) { first = o; break; }
        }
        slot[s] = -first - 1;                                  // for now: who opened my class
        if (first == s) rep[atomicAdd(&s_ncls, 1)] = s;
    }
    __syncthreads();
    const int ncls = s_ncls;
    for (int k = tid; k < ncls; k += kThreads) slot[rep[k]] = k;          // the openers learn their class number
    __syncthreads();
    for (int s = tid; s < S; s += kThreads)
        if (slot[s] < 0) slot[s] = slot[-slot[s] - 1];                    // the others copy it (an opener's entry is final by now)
    const bool vec = (S & 3) == 0;
    __syncthreads();                                            // classes known
    // As many instances at a time as their pair tables fit into the table's room (S * S words; at most S classes):
    // one round of evaluations, one barrier, one run of stores for all of them.
    __shared__ int s_ok[8];
    const int nn = ncls * ncls;
    const int cap = max(1, min(8, (S * S) / max(1, nn)));
    for (int n0 = 0; n0 < inst_per_cta; n0 += cap) {
        const int g = min(cap, inst_per_cta - n0);
        __syncthreads();                                        // the last group's tables are no longer read
        for (int n = 0; n < g; ++n) {
            const int i = cta * inst_per_cta + n0 + n;
            int ok = 0;
            if (i < B) {
                const int Li = L[i];
                ok = Li >= 1 && Li <= Lmax;                     // out of range: nothing written
                if (ok && status) ok = status[i] == 0;          // bad descriptor: already -1
                if (!status) {
                    int bad = 0;
                    if (ok) {
                        bad = s_sbad | (inst_ok(inst[i]) ? 0 : 1);
                        for (int l = tid; l < Li; l += kThreads) bad |= layer_ok(layers[(long long)i * layer_stride_B + l]) ? 0 : 1;
                    }
                    if (__syncthreads_or(bad)) ok = 0;          // flagged: the cost role writes -1 into this matrix too
                }
            }
            if (tid == 0) s_ok[n] = ok;
        }
        __syncthreads();
        for (int e = tid; e < g * nn; e += kThreads) {
            const int n = e / nn, r = e - n * nn;
            if (!s_ok[n]) continue;
            const int i = cta * inst_per_cta + n0 + n;
            const galv_layer_desc ly = layers[(long long)i * layer_stride_B];
            const galv_inst_params in = inst[i];
            const int ka = r / ncls, kc = r - ka * ncls;
            const galv_strategy_desc sa = strat[rep[ka]], sc = strat[rep[kc]];
            const double bq = in.b / sc.batch_div;
            const double bytes = bq * ly.seq * ly.h * in.bytes_per_elem;
            const double t = pair_factor(sa, sc) * bytes / in.bw_tp;
            tab[e] = quant_time(t, in.time_unit_ns);
        }
        __syncthreads();
        for (int n = 0; n < g; ++n) {
            if (!s_ok[n]) continue;
            const int i = cta * inst_per_cta + n0 + n;
            int32_t* const out = trans_q + (size_t)i * S * S;
            const int32_t* const tb = tab + n * nn;
            if (vec) {
                for (int e = tid; e < S * S / 4; e += kThreads) {
                    const int a = (4 * e) / S, c = 4 * e - a * S;
                    const int32_t* row = tb + slot[a] * ncls;
                    reinterpret_cast<int4*>(out)[e] = make_int4(row[slot[c]], row[slot[c + 1]], row[slot[c + 2]], row[slot[c + 3]]);
                }
            } else {
                for (int e = tid; e < S * S; e += kThreads) {
                    const int a = e / S, c = e - a * S;
                    out[e] = tb[slot[a] * ncls + slot[c]];
                }
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads) trans_kernel(int B, int Lmax, int S, const int32_t* __restrict__ L,
                                                         const galv_layer_desc* __restrict__ layers, long long layer_stride_B,
                                                         const galv_strategy_desc* __restrict__ strat,
                                                         const galv_inst_params* __restrict__ inst, const int32_t* __restrict__ status,
                                                         int32_t* __restrict__ trans_q, int inst_per_cta)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    trans_body(blockIdx.x, smem_raw, B, Lmax, S, L, layers, layer_stride_B, strat, inst, status, trans_q, inst_per_cta);
}

__global__ void __launch_bounds__(kThreads) cost_kernel(int Lmax, int S, int KC, const int32_t* __restrict__ L,
                                                        const galv_layer_desc* __restrict__ layers, long long layer_stride_B,
                                                        const galv_strategy_desc* __restrict__ strat,
                                                        const galv_inst_params* __restrict__ inst, double* __restrict__ time_s,
                                                        double* __restrict__ mem_bytes, int32_t* __restrict__ time_q,
                                                        int32_t* __restrict__ mem_q, int32_t* __restrict__ trans_q,
                                                        int32_t* __restrict__ status)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    cost_body(blockIdx.x, smem_raw, Lmax, S, KC, L, layers, layer_stride_B, strat, inst, time_s, mem_bytes, time_q, mem_q, trans_q, status);
}

// The whole cost model in one launch, for batches small enough that a launch counts: the first CTAs write the
// transition matrices (they run longest and check the descriptors for themselves), the others evaluate one
// instance's layers each.  Bandwidth-sized batches take the two kernels one after the other (2 % faster there).
__global__ void __launch_bounds__(kThreads) cost_trans_kernel(int B, int Lmax, int S, int KC, const int32_t* __restrict__ L,
                                                              const galv_layer_desc* __restrict__ layers, long long layer_stride_B,
                                                              const galv_strategy_desc* __restrict__ strat,
                                                              const galv_inst_params* __restrict__ inst, double* __restrict__ time_s,
                                                              double* __restrict__ mem_bytes, int32_t* __restrict__ time_q,
                                                              int32_t* __restrict__ mem_q, int32_t* __restrict__ trans_q,
                                                              int32_t* __restrict__ status, int inst_per_cta)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int tblocks = (int)gridDim.x - B;                      // the transition role first: its CTAs run longest
    if ((int)blockIdx.x >= tblocks)
        cost_body(blockIdx.x - tblocks, smem_raw, Lmax, S, KC, L, layers, layer_stride_B, strat, inst, time_s, mem_bytes, time_q, mem_q, trans_q, status);
    else
        trans_body(blockIdx.x, smem_raw, B, Lmax, S, L, layers, layer_stride_B, strat, inst, nullptr, trans_q, inst_per_cta);
}

// Stacks too long for the per-instance index arrays in shared memory: descriptors checked by one CTA per
// instance, then one thread per element evaluates the expression directly.
__global__ void __launch_bounds__(kThreads) check_kernel(int Lmax, int S, const int32_t* __restrict__ L,
                                                         const galv_layer_desc* __restrict__ layers, long long layer_stride_B,
                                                         const galv_strategy_desc* __restrict__ strat, const galv_inst_params* __restrict__ inst,
                                                         int32_t* __restrict__ time_q, int32_t* __restrict__ mem_q, int32_t* __restrict__ trans_q,
                                                         int32_t* __restrict__ status)
{
    __shared__ int s_bad;
    const int i = blockIdx.x, tid = threadIdx.x;
    const int Li = L[i];
    if (Li < 1 || Li > Lmax) {
        if (tid == 0) status[i] = GALV_STATUS_BAD_INPUT;
        return;
    }
    if (tid == 0) s_bad = inst_ok(inst[i]) ? 0 : 1;
    __syncthreads();
    bool bad = false;
    for (int s = tid; s < S; s += kThreads) bad = bad || !strat_ok(strat[s]);
    for (int l = tid; l < Li; l += kThreads) bad = bad || !layer_ok(layers[(long long)i * layer_stride_B + l]);
    if (bad) atomicOr(&s_bad, 1);
    __syncthreads();
    if (tid == 0) status[i] = s_bad ? GALV_STATUS_BAD_INPUT : 0;
    if (s_bad) {
        const size_t base = (size_t)i * Lmax * S;
        for (int e = tid; e < Li * S; e += kThreads) { time_q[base + e] = -1; mem_q[base + e] = -1; }
        for (int e = tid; e < S * S; e += kThreads) trans_q[(size_t)i * S * S + e] = -1;
    }
}

__global__ void cost_direct_kernel(int B, int Lmax, int S, const int32_t* __restrict__ L, const galv_layer_desc* __restrict__ layers,
                                   long long layer_stride_B, const galv_strategy_desc* __restrict__ strat,
                                   const galv_inst_params* __restrict__ inst, const int32_t* __restrict__ status,
                                   double* __restrict__ time_s, double* __restrict__ mem_bytes, int32_t* __restrict__ time_q,
                                   int32_t* __restrict__ mem_q)
{
    const long long n = (long long)B * Lmax * S;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
        const int s = (int)(e % S);
        const long long il = e / S;
        const int l = (int)(il % Lmax), i = (int)(il / Lmax);
        const int Li = L[i];
        if (Li < 1 || Li > Lmax || l >= Li || status[i] != 0) continue;
        const galv_inst_params in = inst[i];
        double t, b;
        cost_of(layers[(long long)i * layer_stride_B + l], strat[s], in, &t, &b);
        if (time_s) time_s[e] = t;
        if (mem_bytes) mem_bytes[e] = b;
        time_q[e] = quant_time(t, in.time_unit_ns);
        mem_q[e] = quant_mem(b, in.bin_bytes);
    }
}

}  // namespace

cudaError_t galv_costs_launch(const galv_shape* sh, const int32_t* L, const galv_layer_desc* layers,
                              int64_t layer_stride_B, const galv_strategy_desc* strat,
                              const galv_inst_params* inst, double* time_s, double* mem_bytes,
                              int32_t* time_q, int32_t* mem_q, int32_t* trans_q, int32_t* status,
                              cudaStream_t st)
{
    const int S = sh->S, Lmax = sh->Lmax;
    const bool want_d = time_s != nullptr || mem_bytes != nullptr;
    // instances per CTA of the transition role: the pair-factor table is worth sharing only when CTAs are plenty
    int ipc = sh->B / (2 * 148);
    ipc = ipc < 1 ? 1 : (ipc > 8 ? 8 : ipc);
    const int tblocks = (sh->B + ipc - 1) / ipc;
    const size_t tsmem = ((size_t)2 * S + (size_t)S * S) * 4;          // at most S classes
    // distinct layers evaluated per pass: as many as fit beside the layer index arrays in 40 KB
    const size_t fixed = (size_t)(3 * Lmax + 4) * 4;
    const size_t per_kind = (size_t)S * (want_d ? 24 : 8);
    const size_t budget = 40 * 1024;
    if (fixed + per_kind + 16 > 200 * 1024) {
        // very long stacks: no room for the layer index arrays; descriptors checked first, then one thread per element,
        // then the transition matrices of the instances that passed
        check_kernel<<<sh->B, kThreads, 0, st>>>(Lmax, S, L, layers, (long long)layer_stride_B, strat, inst, time_q, mem_q, trans_q, status);
        const long long n = (long long)sh->B * Lmax * S;
        long long blocks = (n + 255) / 256;
        if (blocks > 148 * 16) blocks = 148 * 16;
        cost_direct_kernel<<<(int)blocks, 256, 0, st>>>(sh->B, Lmax, S, L, layers, (long long)layer_stride_B, strat, inst, status, time_s, mem_bytes,
                                                        time_q, mem_q);
        if (tsmem > 48 * 1024) {                                   // long stacks or many strategies only; per device, so asked every time
            cudaError_t e = cudaFuncSetAttribute(trans_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tsmem);
            if (e != cudaSuccess) return e;
        }
        trans_kernel<<<tblocks, kThreads, tsmem, st>>>(sh->B, Lmax, S, L, layers, (long long)layer_stride_B, strat, inst, status, trans_q, ipc);
        return cudaGetLastError();
    }
    size_t smem;
    int kc;
    if (fixed + per_kind + 16 > budget) {
        // long stacks: the index arrays alone pass 40 KB; one distinct layer per pass
        kc = 1;
        smem = fixed + per_kind + 16;
    } else {
        kc = (int)((budget - fixed - 16) / per_kind);
        if (kc > Lmax) kc = Lmax;
        smem = fixed + (size_t)kc * per_kind + 16;
    }
    if (sh->B > 1024) {
        if (smem > 48 * 1024) {                                   // long stacks or many strategies only; per device, so asked every time
            cudaError_t e = cudaFuncSetAttribute(cost_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
        }
        cost_kernel<<<sh->B, kThreads, smem, st>>>(Lmax, S, kc, L, layers, (long long)layer_stride_B, strat, inst, time_s, mem_bytes, time_q,
                                                   mem_q, trans_q, status);
        if (tsmem > 48 * 1024) {                                   // long stacks or many strategies only; per device, so asked every time
            cudaError_t e = cudaFuncSetAttribute(trans_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tsmem);
            if (e != cudaSuccess) return e;
        }
        trans_kernel<<<tblocks, kThreads, tsmem, st>>>(sh->B, Lmax, S, L, layers, (long long)layer_stride_B, strat, inst, status, trans_q, ipc);
        return cudaGetLastError();
    }
    if (tsmem > smem) smem = tsmem;                                   // one launch, two roles: the larger of their needs
    if (smem > 48 * 1024) {                                   // long stacks or many strategies only; per device, so asked every time
        cudaError_t e = cudaFuncSetAttribute(cost_trans_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    cost_trans_kernel<<<sh->B + tblocks, kThreads, smem, st>>>(sh->B, Lmax, S, kc, L, layers, (long long)layer_stride_B, strat, inst, time_s,
                                                              mem_bytes, time_q, mem_q, trans_q, status, ipc);
    return cudaGetLastError();
}
