// Outer selection over the instance batch: per group of candidates (micro-batch, pipeline degree)
// the one with the shortest pipeline iteration, (n_micro + pp - 1) * stage optimum.
// (Section 3 of the paper: the plan also fixes pipeline stages and micro-batch.)
// A segmented (min, then lowest index) reduction over B <= a few thousand values: two tiny
// passes with 64-bit and 32-bit atomic minima; launch-latency bound.

#include "galv_internal.h"

namespace {

constexpr unsigned long long kNone = ~0ull;

__device__ __forceinline__ bool candidate(int i, int G, const int32_t* opt_cost, const int32_t* status,
                                          const int32_t* n_micro, const int32_t* pp, const int32_t* group,
                                          unsigned long long* t)
{
    const int c = opt_cost[i];
    if (status[i] != 0 || c >= GALV_INF || c < 0) return false;
    if (n_micro[i] < 1 || pp[i] < 1 || group[i] < 0 || group[i] >= G) return false;
    *t = (unsigned long long)((long long)n_micro[i] + pp[i] - 1) * (unsigned long long)c;
    return true;
}

__global__ void select_init_kernel(int G, unsigned long long* best_time, int32_t* best_inst)
{
    for (int g = blockIdx.x * blockDim.x + threadIdx.x; g < G; g += gridDim.x * blockDim.x) {
        best_time[g] = kNone;
        best_inst[g] = 0x7fffffff;
    }
}

__global__ void select_time_kernel(int B, int G, const int32_t* opt_cost, const int32_t* status, const int32_t* n_micro,
                                   const int32_t* pp, const int32_t* group, unsigned long long* best_time)
{
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < B; i += gridDim.x * blockDim.x) {
        unsigned long long t;
        if (candidate(i, G, opt_cost, status, n_micro, pp, group, &t)) atomicMin(&best_time[group[i]], t);
    }
}

__global__ void select_inst_kernel(int B, int G, const int32_t* opt_cost, const int32_t* status, const int32_t* n_micro,
                                   const int32_t* pp, const int32_t* group, const unsigned long long* best_time,
                                   int32_t* best_inst)
{
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < B; i += gridDim.x * blockDim.x) {
        unsigned long long t;
        if (candidate(i, G, opt_cost, status, n_micro, pp, group, &t) && t == best_time[group[i]])
            atomicMin(&best_inst[group[i]], i);
    }
}

__global__ void select_finish_kernel(int G, long long* best_time, int32_t* best_inst)
{
    for (int g = blockIdx.x * blockDim.x + threadIdx.x; g < G; g += gridDim.x * blockDim.x)
        if (best_inst[g] == 0x7fffffff) { best_time[g] = -1; best_inst[g] = -1; }
}

}  // namespace

extern "C" int galv_select_best(galv_ctx* ctx, int32_t B, int32_t G, const int32_t* opt_cost, const int32_t* status,
                                const int32_t* n_micro, const int32_t* pp, const int32_t* group,
                                int64_t* best_time, int32_t* best_inst, void* stream)
{
    if (!ctx) return GALV_ERR_INVALID_ARG;
    if (B < 1 || G < 1 || !opt_cost || !status || !n_micro || !pp || !group || !best_time || !best_inst)
        return galv_set_error(ctx, GALV_ERR_INVALID_ARG, "galv_select_best: B, G >= 1 and no NULL pointer");
    cudaStream_t st = (cudaStream_t)stream;
    const int gb = (G + 255) / 256 > 1024 ? 1024 : (G + 255) / 256, bb = (B + 255) / 256 > 1024 ? 1024 : (B + 255) / 256;
    unsigned long long* bt = reinterpret_cast<unsigned long long*>(best_time);
    select_init_kernel<<<gb, 256, 0, st>>>(G, bt, best_inst);
    select_time_kernel<<<bb, 256, 0, st>>>(B, G, opt_cost, status, n_micro, pp, group, bt);
    select_inst_kernel<<<bb, 256, 0, st>>>(B, G, opt_cost, status, n_micro, pp, group, bt, best_inst);
    select_finish_kernel<<<gb, 256, 0, st>>>(G, reinterpret_cast<long long*>(best_time), best_inst);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? GALV_OK : galv_set_error(ctx, GALV_ERR_CUDA, cudaGetErrorString(e));
}
