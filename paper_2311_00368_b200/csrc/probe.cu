// Measurement aids, not part of the method: the FP32 FMA rate this GPU sustains right now (register-only FMA
// chains on every SM), for the denominator of the roofline fraction; and the rate at which an SM pulls operand
// tiles out of L2 into shared memory with bulk asynchronous copies, the second resource the dense-tile kernels
// load heavily.
#include <cuda_runtime.h>
#include <stdint.h>

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

constexpr int kPullChunk = 32768;   // bytes per copy: the dense-tile kernels' pipeline chunk
constexpr int kPullDepth = 3;       // copies in flight per CTA: their ring

__device__ __forceinline__ uint32_t shared_addr(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

// One CTA per SM; thread 0 keeps kPullDepth bulk copies of kPullChunk bytes in flight from `src` (walked with a
// stride so that neighbouring CTAs read different lines) and waits for each on an mbarrier, with a limit: a wait
// that runs out sets sink[1] and ends the CTA's loop after its copies in flight have had the same limit to land.
__global__ void __launch_bounds__(128, 1) l2_pull_kernel(const char *src, size_t bytes, int iters, unsigned long long *sink)
{
    extern __shared__ __align__(1024) char buf[];
    __shared__ __align__(8) unsigned long long bar[kPullDepth];
    if (threadIdx.x == 0) {
        for (int i = 0; i < kPullDepth; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(shared_addr(&bar[i])));
        asm volatile("fence.mbarrier_init.release.cluster;");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const size_t nchunks = bytes / kPullChunk;
        size_t pos = (size_t)blockIdx.x * 977 % nchunks;
        bool gave_up = false;
        int drain = kPullDepth - 1;   // after a wait has run out: this many more waits, for the copies still in flight
        for (int it = 0; it < iters + kPullDepth; ++it) {
            const int s = it % kPullDepth;
            if (it >= kPullDepth) {
                const uint32_t parity = ((it / kPullDepth) - 1) & 1;
                uint32_t done = 0;
                for (int spin = 0; spin < (1 << 22) && !done; ++spin)
                    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                                 : "=r"(done) : "r"(shared_addr(&bar[s])), "r"(parity) : "memory");
                if (!done) gave_up = true;
            }
            if (gave_up) {
                if (drain-- <= 0) break;
                continue;
            }
            if (it < iters) {
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(shared_addr(&bar[s])), "r"(kPullChunk) : "memory");
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(shared_addr(buf + (size_t)s * kPullChunk)), "l"(src + pos * kPullChunk), "r"(kPullChunk),
                               "r"(shared_addr(&bar[s])) : "memory");
                pos = (pos + 131) % nchunks;
            }
        }
        if (gave_up) sink[1] = 1;
    }
    __syncthreads();
    if (threadIdx.x == 0 && buf[0] == 123 && buf[kPullChunk] == 45) sink[0] = 1;   // keeps the copies observable; practically never true
}

}  // namespace

extern "C" b2sp_status b2sp_probe_l2_pull(void *scratch, size_t scratch_bytes, double *gbs_per_sm_host, double *gbs_total_host, void *stream)
{
    if (!scratch || scratch_bytes < (size_t)(1 << 20) + 16 || !gbs_per_sm_host || !gbs_total_host) return B2SP_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(scratch) & 15) return B2SP_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return B2SP_ERR_CUDA;
    // the first 16 bytes are the kernel's two result words, the rest (whole chunks, at most 16 MB so that it stays in L2) the source
    unsigned long long *sink = static_cast<unsigned long long *>(scratch);
    const char *src = static_cast<const char *>(scratch) + kPullChunk;
    size_t bytes = (scratch_bytes - kPullChunk) / kPullChunk * kPullChunk;
    if (bytes > ((size_t)16 << 20)) bytes = (size_t)16 << 20;
    const int smem = kPullDepth * kPullChunk;
    if (cudaFuncSetAttribute(l2_pull_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return B2SP_ERR_CUDA;
    if (cudaMemsetAsync(scratch, 0, 16, st) != cudaSuccess) return B2SP_ERR_CUDA;
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess) return B2SP_ERR_CUDA;
    if (cudaEventCreate(&e1) != cudaSuccess) { cudaEventDestroy(e0); return B2SP_ERR_CUDA; }
    const int iters = 2000;
    double best = 0.0;
    b2sp_status rc = B2SP_OK;
    for (int rep = 0; rep < 6 && rc == B2SP_OK; ++rep) {   // first launch warms up (and brings the source into L2); best of 5
        cudaEventRecord(e0, st);
        l2_pull_kernel<<<sms, 128, smem, st>>>(src, bytes, iters, sink);
        cudaEventRecord(e1, st);
        float ms = 0.f;
        if (cudaEventSynchronize(e1) != cudaSuccess || cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess ||
            cudaGetLastError() != cudaSuccess) {
            rc = B2SP_ERR_CUDA;
            break;
        }
        const double gbs = (double)iters * kPullChunk / (ms * 1e6);
        if (rep > 0 && ms > 0.f && gbs > best) best = gbs;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    unsigned long long words[2] = {0, 0};
    if (rc == B2SP_OK && cudaMemcpyAsync(words, sink, sizeof(words), cudaMemcpyDeviceToHost, st) != cudaSuccess) rc = B2SP_ERR_CUDA;
    if (rc == B2SP_OK && cudaStreamSynchronize(st) != cudaSuccess) rc = B2SP_ERR_CUDA;
    if (rc == B2SP_OK && words[1]) rc = B2SP_ERR_TIMEOUT;
    *gbs_per_sm_host = best;
    *gbs_total_host = best * sms;
    return rc;
}

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
