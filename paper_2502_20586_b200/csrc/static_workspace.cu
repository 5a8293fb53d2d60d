// mxfp4_linear_backward_static: the linear-layer backward for callers that cannot obtain device scratch memory.
//
// mxfp4_linear_backward needs a workspace for the quantised operands, which its caller normally takes from its
// own allocator.  Some callers have no allocator to turn to at the point of the call: a hook that runs while the
// host framework's memory pool is locked or already handed out in full, a plug-in that is forbidden to touch the
// CUDA allocator of the process that hosts it, a tool that must keep working after device memory has been
// exhausted.  For them the scratch lives in the library image itself: a fixed array in device global memory that
// every GPU which loads this library carries from load to exit (MXFP4_STATIC_WORKSPACE_BYTES per GPU).
//
// Nothing in this file allocates: no cudaMalloc / cudaFree, no allocating library routine.
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "../../include/mxfp4.h"

namespace {

// The scratch itself.  In host code this name is only a stand-in for the symbol: it is NOT a device address and
// must never be handed to a kernel; the address is asked for once per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_workspace[MXFP4_STATIC_WORKSPACE_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_workspace_ptr[kMaxDevices] = {};     // per device: device address of g_static_workspace, or nullptr

// Device address of the scratch array on the CURRENT device; looked up on the first call per device.
mxfp4_status static_workspace(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return MXFP4_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return MXFP4_ERR_DEVICE;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_workspace_ptr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_workspace) != cudaSuccess || ptr == nullptr) return MXFP4_ERR_CUDA;
        g_workspace_ptr[dev] = ptr;
    }
    *out = g_workspace_ptr[dev];
    return MXFP4_OK;
}

}  // namespace

extern "C" mxfp4_status mxfp4_linear_backward_static(const void* dY, const void* X, const void* W, int64_t b, int64_t m, int64_t n,
                                                     int g, int rounding, uint64_t seed, void* dX, void* dW, int out_dtype,
                                                     void* cuda_stream) {
    if (b <= 0 || m <= 0 || n <= 0) return MXFP4_ERR_SHAPE;
    const size_t need = mxfp4_linear_backward_workspace(b, m, n);
    if (need == 0 || need > (size_t)MXFP4_STATIC_WORKSPACE_BYTES) return MXFP4_ERR_WORKSPACE;   // shapes too large for the fixed scratch
    void* ws = nullptr;
    const mxfp4_status st = static_workspace(&ws);
    if (st != MXFP4_OK) return st;
    // Every byte the GEMMs read from the scratch is rewritten by this call's quantisers first, so nothing has to be
    // cleared; bytes a call does not write (padding of the scale tiles) only feed outputs that are never stored.
    return mxfp4_linear_backward(dY, X, W, b, m, n, g, rounding, seed, dX, dW, out_dtype, ws, (size_t)MXFP4_STATIC_WORKSPACE_BYTES, cuda_stream);
}
