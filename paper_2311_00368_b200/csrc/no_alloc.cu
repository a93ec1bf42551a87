// b2sp_spmm_static_scratch: SPMM for callers that cannot allocate device memory.
//
// Some users of this library run where cudaMalloc is off limits: a plug-in inside an inference
// server whose host process handed every byte of device memory to its own arena at start-up, or a
// latency-critical loop that cannot afford the device-wide synchronisation an allocation may
// cause.  Such a caller can supply inputs and outputs (they come from the host's arena) but has
// nowhere to get the row-binning workspace the regular entry point asks for.  This file gives
// that workspace a permanent home: a fixed array in the library's own device image.
//
// The array is part of the library's device image and costs kScratchBytes of device memory on every
// GPU where that image gets loaded, until the process exits.  With CUDA's lazy module loading the
// first cudaGetSymbolAddress on a device is what loads the image there: the driver reserves the
// array (and the code) at that moment and may synchronise the device.  That first call therefore
// belongs at start-up, before the host's arena takes the rest of the memory.
#include "../../include/b2sp.h"

#include <cuda_runtime.h>

#include <mutex>

namespace {

constexpr int kMaxRows = B2SP_STATIC_SCRATCH_MAX_ROWS;
// 512-byte header (histogram, cursors, status words) + one int per row, as b2sp_workspace_bytes
// lays the workspace out.
constexpr size_t kScratchBytes = 512 + sizeof(int) * (size_t)kMaxRows;

// In host code the name `g_scratch` is only a handle for the runtime to look the array up by;
// it is NOT the array's device address and must never be handed to a kernel.  The address the
// kernels need is what cudaGetSymbolAddress returns, per device.
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void *g_scratch_addr[kMaxDevices] = {};

// Resolves the array's address on the current device the first time that device is seen.
b2sp_status scratch_for_current_device(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return B2SP_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return B2SP_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return B2SP_ERR_CUDA;
        }
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return B2SP_OK;
}

}  // namespace

extern "C" b2sp_status b2sp_spmm_static_scratch(int M, int K, int N, long long nnz, const int *row_ptr,
                                                const int *col_idx, const float *values,
                                                const float *D, long long ldd, float *O,
                                                long long ldo, void *stream)
{
    if (M > kMaxRows) return B2SP_ERR_TOO_LARGE;
    void *scratch = nullptr;
    b2sp_status rc = scratch_for_current_device(&scratch);
    if (rc != B2SP_OK) return rc;
    // The row family only enqueues a memset of the scratch header and kernels; it never allocates.
    // Everything in the scratch that has to start from zero (histogram, cursors, status) is in
    // that header and is cleared at the start of every call; row_order[0..M) is fully rewritten.
    return b2sp_spmm(M, K, N, nnz, row_ptr, col_idx, values, D, ldd, O, ldo, scratch, kScratchBytes,
                     B2SP_ALGO_ROW, stream);
}
