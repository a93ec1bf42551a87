// Measurement aid: the FP32 FMA rate this GPU sustains right now (register-only FMA chains on every
// SM), for the denominator of the roofline fraction.  Not part of the method.
#include <cuda_runtime.h>

#include "../../include/b2sp_debug.h"

namespace {

constexpr int kChains = 8;       // independent accumulators per thread (FMA latency ~4 cycles, 4 schedulers)
constexpr int kThreads = 256;
constexpr int kBlocksPerSM = 8;  // 2048 threads per SM

__global__ void __launch_bounds__(kThreads) fma_chain_kernel(int iters, float seed, float *sink)
{
    float acc[kChains];
#pragma unroll
    for (int c = 0; c < kChains; ++c) acc[c] = seed + (float)(threadIdx.x + c);
    const float m = 1.0000001f, add = 1e-7f;
    for (int i = 0; i < iters; ++i) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
#pragma unroll
            for (int c = 0; c < kChains; ++c) acc[c] = fmaf(acc[c], m, add);
        }
    }
    float s = 0.f;
#pragma unroll
    for (int c = 0; c < kChains; ++c) s += acc[c];
    if (s == 123.456f) sink[0] = s;   // keeps the chains alive; practically never true
}

}  // namespace

extern "C" b2sp_status b2sp_probe_fp32_peak(int iters, float *scratch, double *gflops_host, void *stream)
{
    if (iters <= 0 || !scratch || !gflops_host) return B2SP_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return B2SP_ERR_CUDA;
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess) return B2SP_ERR_CUDA;
    if (cudaEventCreate(&e1) != cudaSuccess) { cudaEventDestroy(e0); return B2SP_ERR_CUDA; }
    const int blocks = sms * kBlocksPerSM;
    double best = 0.0;
    b2sp_status rc = B2SP_OK;
    for (int rep = 0; rep < 11 && rc == B2SP_OK; ++rep) {   // first launch warms up; best of 10
        cudaEventRecord(e0, st);
        fma_chain_kernel<<<blocks, kThreads, 0, st>>>(iters, 1.0f, scratch);
        cudaEventRecord(e1, st);
        float ms = 0.f;
        if (cudaEventSynchronize(e1) != cudaSuccess || cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess ||
            cudaGetLastError() != cudaSuccess) {
            rc = B2SP_ERR_CUDA;
            break;
        }
        const double flops = 2.0 * kChains * 8.0 * (double)iters * kThreads * (double)blocks;
        if (rep > 0 && ms > 0.f && flops / (ms * 1e6) > best) best = flops / (ms * 1e6);
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    *gflops_host = best;
    return rc;
}
