// galv_dp_search_static: the search for callers that cannot hand over a workspace.
//
// Same kernels as galv_dp_search; the scratch (instance order, per-layer activity counts, the
// device error flag, and the two-layer rolling buffer when the full table is not kept) lives in a
// fixed array in this library's device image instead of memory the caller allocates.

#include <mutex>

#include "galv_internal.h"

namespace {

// One copy per GPU that loads the library, held until the process exits.
__device__ __align__(256) unsigned char g_static_workspace[GALV_STATIC_WORKSPACE_BYTES];

constexpr int kMaxDevices = 64;
void* g_workspace_addr[kMaxDevices];        // device address of g_static_workspace, per device ordinal
std::mutex g_setup_mutex;

// In host code `g_static_workspace` names a host-side shadow of the symbol, not device memory;
// the address a kernel may use has to be asked for, once per device, with that device current.
cudaError_t workspace_address(int device, void** out)
{
    if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_workspace_addr[device]) {
        int cur = -1;
        cudaError_t e = cudaGetDevice(&cur);
        if (e != cudaSuccess) return e;
        if (cur != device && (e = cudaSetDevice(device)) != cudaSuccess) return e;
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_workspace);
        if (cur != device) cudaSetDevice(cur);
        if (e != cudaSuccess) return e;
        g_workspace_addr[device] = p;
    }
    *out = g_workspace_addr[device];
    return cudaSuccess;
}

}  // namespace

extern "C" int galv_dp_search_static(galv_ctx* ctx, const galv_shape* sh, const int32_t* L, const int32_t* time_q,
                                     const int32_t* mem_q, const int32_t* trans_q, int32_t* C, uint8_t* A,
                                     int32_t* C_last, int32_t* status, void* stream)
{
    if (!ctx) return GALV_ERR_INVALID_ARG;
    const size_t need = galv_dp_workspace_bytes(ctx, sh);
    if (need == 0) return galv_set_error(ctx, GALV_ERR_INVALID_ARG, "galv_dp_search_static: shape outside limits");
    if (need > (size_t)GALV_STATIC_WORKSPACE_BYTES)
        return galv_set_error(ctx, GALV_ERR_WORKSPACE,
                              "galv_dp_search_static: this shape needs more scratch than the built-in "
                              "GALV_STATIC_WORKSPACE_BYTES; use galv_dp_search with a workspace");
    void* ws = nullptr;
    const cudaError_t e = workspace_address(ctx->device, &ws);
    if (e != cudaSuccess) return galv_set_error(ctx, GALV_ERR_CUDA, cudaGetErrorString(e));
    return galv_dp_search(ctx, sh, L, time_q, mem_q, trans_q, C, A, C_last, ws, GALV_STATIC_WORKSPACE_BYTES, status, stream);
}
