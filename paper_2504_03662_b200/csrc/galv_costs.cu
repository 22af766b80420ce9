// Cost model of the strategy search: fp64, elementwise, one thread per output.
//
// (Section 3 of the paper: the selector builds a performance model from the
// model profiler's per-layer shapes and FLOPs, the hardware profiler's memory
// and link bandwidth, and the dataset profiler's batch.)
//
// This translation unit is compiled with -fmad=false: every product and sum is
// rounded on its own, in the order written, so the doubles equal what any IEEE
// host computes from the same expression tree.  Outputs are [B][Lmax][S] with s
// fastest: consecutive threads write consecutive addresses (coalesced); the
// descriptor reads are warp-broadcast loads through the read-only path.

#include "galv_internal.h"

namespace {

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

struct Desc10 { double v[10]; };

__global__ void cost_kernel(int B, int Lmax, int S, const int32_t* __restrict__ L,
                            const galv_layer_desc* __restrict__ layers, long long layer_stride_B,
                            const galv_strategy_desc* __restrict__ strat, const galv_inst_params* __restrict__ inst,
                            double* __restrict__ time_s, double* __restrict__ mem_bytes,
                            int32_t* __restrict__ time_q, int32_t* __restrict__ mem_q, int32_t* __restrict__ status)
{
    const long long n = (long long)B * Lmax * S;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
        const int s = (int)(e % S);
        const long long il = e / S;
        const int l = (int)(il % Lmax);
        const int i = (int)(il / Lmax);
        const int Li = __ldg(L + i);
        if (Li < 1 || Li > Lmax) {
            if (l == 0 && s == 0) status[i] = GALV_STATUS_BAD_INPUT;
            continue;
        }
        if (l == 0 && s == 0) status[i] = 0;
        if (l >= Li) continue;
        const galv_layer_desc ly = layers[(long long)i * layer_stride_B + l];
        const galv_strategy_desc sd = strat[s];
        const galv_inst_params in = inst[i];

        const double tp = (double)sd.tp, dp = (double)sd.dp;
        const double bq = in.b / sd.batch_div;
        const double sbh = ly.seq * bq * ly.h;
        const double fwd = ly.c_lin * bq * ly.seq * ly.h * ly.h + ly.c_attn * bq * ly.seq * ly.seq * ly.h;
        const double t_comp = fwd * (3.0 + (double)sd.ckpt) / tp / in.flops_rate;
        const double t_tp = ly.n_ar * (2.0 * (tp - 1.0) / tp) * (bq * ly.seq * ly.h * in.bytes_per_elem) / in.bw_tp;
        const double zmul = sd.zero == 3 ? 1.5 : 1.0;
        const double t_dp = zmul * (2.0 * (dp - 1.0) / dp) * (ly.p_coef * ly.h * ly.h * in.bytes_per_elem / tp) / in.bw_dp;
        const double t = (t_comp + t_tp) + t_dp;

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
        const double mb = state + in.act_mult * act;

        if (time_s) time_s[e] = t;
        if (mem_bytes) mem_bytes[e] = mb;
        time_q[e] = quant_time(t, in.time_unit_ns);
        mem_q[e] = quant_mem(mb, in.bin_bytes);
    }
}

// trans_q[i][a][c]: resharding time from strategy a (previous layer) to c (this layer).
__global__ void trans_kernel(int B, int Lmax, int S, const int32_t* __restrict__ L,
                             const galv_layer_desc* __restrict__ layers, long long layer_stride_B,
                             const galv_strategy_desc* __restrict__ strat, const galv_inst_params* __restrict__ inst,
                             int32_t* __restrict__ trans_q)
{
    const long long n = (long long)B * S * S;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(e % S);
        const long long ia = e / S;
        const int a = (int)(ia % S);
        const int i = (int)(ia / S);
        const int Li = __ldg(L + i);
        if (Li < 1 || Li > Lmax) continue;
        const galv_layer_desc ly = layers[(long long)i * layer_stride_B];
        const galv_strategy_desc sa = strat[a], sc = strat[c];
        const galv_inst_params in = inst[i];
        const double tpa = (double)sa.tp, tpc = (double)sc.tp;
        const double bq = in.b / sc.batch_div;
        const double bytes = bq * ly.seq * ly.h * in.bytes_per_elem;
        const double k = (tpa > tpc ? tpa : tpc) / (tpa < tpc ? tpa : tpc);
        const double spterm = (sa.sp != sc.sp) ? (tpc - 1.0) / tpc : 0.0;
        const double t = ((k - 1.0) / k + spterm) * bytes / in.bw_tp;
        trans_q[e] = quant_time(t, in.time_unit_ns);
    }
}

}  // namespace

cudaError_t galv_costs_launch(const galv_shape* sh, const int32_t* L, const galv_layer_desc* layers,
                              int64_t layer_stride_B, const galv_strategy_desc* strat,
                              const galv_inst_params* inst, double* time_s, double* mem_bytes,
                              int32_t* time_q, int32_t* mem_q, int32_t* trans_q, int32_t* status,
                              cudaStream_t st)
{
    const long long n = (long long)sh->B * sh->Lmax * sh->S;
    long long blocks = (n + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    cost_kernel<<<(int)blocks, 256, 0, st>>>(sh->B, sh->Lmax, sh->S, L, layers, (long long)layer_stride_B, strat, inst,
                                             time_s, mem_bytes, time_q, mem_q, status);
    const long long nt = (long long)sh->B * sh->S * sh->S;
    blocks = (nt + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    trans_kernel<<<(int)blocks, 256, 0, st>>>(sh->B, sh->Lmax, sh->S, L, layers, (long long)layer_stride_B, strat, inst, trans_q);
    return cudaGetLastError();
}
