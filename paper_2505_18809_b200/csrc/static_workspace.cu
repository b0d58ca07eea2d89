// vorta_routed_attention_static: the routed-attention layer for callers that cannot
// allocate device memory.  The scratch the core-set branch needs (index list, scatter
// map, gathered Q/K/V, compact output) lives in a fixed array that is part of the
// library image instead of a caller-provided workspace.
#include <mutex>

#include "vorta_internal.h"

namespace {

// Scratch of the core-set branch.  Every device that loads the library carries these
// bytes from load until the process ends, so the size is kept modest.
__device__ __align__(256) unsigned char g_static_workspace[VORTA_STATIC_WORKSPACE_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void *g_workspace_ptr[kMaxDevices] = {};  // device address of the array, per device

// In host code `g_static_workspace` is only a handle for the symbol, not an address a
// kernel may use; the device address has to be asked for, once per device, with that
// device current.
int workspace_address(int device, void **out)
{
    if (device < 0 || device >= kMaxDevices) return VORTA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_workspace_ptr[device]) {
        int prev = -1;
        if (cudaGetDevice(&prev) != cudaSuccess) return VORTA_ERR_CUDA;
        if (prev != device && cudaSetDevice(device) != cudaSuccess) return VORTA_ERR_CUDA;
        void *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_workspace);
        if (prev != device) cudaSetDevice(prev);
        if (e != cudaSuccess || !ptr) {
            cudaGetLastError();
            return VORTA_ERR_CUDA;
        }
        g_workspace_ptr[device] = ptr;
    }
    *out = g_workspace_ptr[device];
    return VORTA_OK;
}

}  // namespace

extern "C" int vorta_routed_attention_static(const vorta_plan *plan, const void *Q, const void *K, const void *V,
                                             void *O, const void *X_or_null, int32_t Hx, void *stream)
{
    if (!plan) return VORTA_ERR_INVALID_ARG;
    vorta_plan_info_t info;
    int rc = vorta_plan_info(plan, &info);
    if (rc != VORTA_OK) return rc;
    if (info.workspace_bytes > (int64_t)VORTA_STATIC_WORKSPACE_BYTES) return VORTA_ERR_WORKSPACE;
    int device = -1;
    rc = vorta_plan_device(plan, &device);
    if (rc != VORTA_OK) return rc;
    void *ws = nullptr;
    rc = workspace_address(device, &ws);
    if (rc != VORTA_OK) return rc;
    return vorta_routed_attention(plan, Q, K, V, O, X_or_null, Hx, ws, (size_t)VORTA_STATIC_WORKSPACE_BYTES, stream);
}
