// Integer-ALU throughput probe: the measured denominator of the ALU roofline.
// Register-only kernel, 32 independent dependency chains per thread, every SM
// filled with resident warps.  Not part of the search path.

#include "galv_internal.h"

namespace {

__device__ int g_probe_sink;

template <int KIND>
__global__ void __launch_bounds__(256) probe_kernel(int iters, int seed)
{
    int acc[32], t[8], c[4];
#pragma unroll
    for (int k = 0; k < 32; ++k) acc[k] = seed + (threadIdx.x ^ (k * 37));
#pragma unroll
    for (int k = 0; k < 8; ++k) t[k] = (seed >> k) - 3 + k + (int)blockIdx.x;
#pragma unroll
    for (int k = 0; k < 4; ++k) c[k] = seed * (k + 5) + (int)threadIdx.x;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                int& a = acc[j * 8 + u];
                if (KIND == 0) a = __viaddmin_s32(a, t[u], c[j]);          // one instruction per relaxation
                else if (KIND == 1) { int v = a + t[u]; a = v < c[j] ? v : c[j]; }   // as the compiler lowers it
                else if (KIND == 2) a = (a + t[u]) ^ c[j];                  // two plain integer operations
                else if (KIND == 3) a = (int)__viaddmin_u16x2((unsigned)c[j], (unsigned)t[u], (unsigned)a);   // packed 16-bit pair: two relaxations
                else a = __vimin3_s32(a, t[u], c[j]);                       // three-input minimum (side work of the packed loop)
            }
    }
    int r = 0;
#pragma unroll
    for (int k = 0; k < 32; ++k) r ^= acc[k];
    if (r == 0x5a5a5a5a && iters < 0) g_probe_sink = r;      // keeps the chains alive; never true
}

}  // namespace

cudaError_t galv_probe_launch(const galv_ctx* ctx, int kind, int iters, int32_t*, cudaStream_t st, long long* ops)
{
    const int blocks = ctx->num_sms * 8, threads = 256;
    if (kind == 0) probe_kernel<0><<<blocks, threads, 0, st>>>(iters, 12345);
    else if (kind == 1) probe_kernel<1><<<blocks, threads, 0, st>>>(iters, 12345);
    else if (kind == 2) probe_kernel<2><<<blocks, threads, 0, st>>>(iters, 12345);
    else if (kind == 3) probe_kernel<3><<<blocks, threads, 0, st>>>(iters, 12345);
    else probe_kernel<4><<<blocks, threads, 0, st>>>(iters, 12345);
    // kinds 0 and 1 count relaxations (add+min pairs); kind 2 counts both of its operations; kind 3 counts the
    // two relaxations each packed instruction performs; kind 4 counts instructions
    *ops = (long long)blocks * threads * 32 * iters * ((kind == 2 || kind == 3) ? 2 : 1);
    return cudaGetLastError();
}
