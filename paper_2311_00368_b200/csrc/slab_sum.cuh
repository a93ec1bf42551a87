// Several partial outputs ("slabs") per output tile of the dense-tile FusedMM / SPMM -- one per K split, or one per
// segment of the balanced partition -- and the kernel that adds them, always in slab order, into O.
//
// The tile kernel's CTAs end at about the same time, so a CTA that summed its tile inside that kernel did it with
// one SM while the others were already idle (measured: 5% of an SPMM on 8192^2, 12% with the balanced partition).
// slab_sum_kernel, a programmatic dependent of the tile kernel, does it with the whole GPU, from L2.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace b2sp {

constexpr int kSlabTileRows = 128;   // rows of an output tile (= kFusedRows)

// The balanced partition deals the granules of all row tiles evenly to groups of CTAs: group c of n gets granules
// [c * G / n, (c + 1) * G / n) of G.  In 32-bit arithmetic throughout (G < 2^31, n a few hundred at most): 64-bit
// divisions are calls of a library routine, and a call in the tile kernel cost it 9% of its speed.
struct Balance {
    int gtot, groups, q, r;   // G, n, G / n, G % n
    __host__ __device__ Balance(int gtot_, int groups_) : gtot(gtot_), groups(groups_), q(gtot_ / groups_), r(gtot_ % groups_) {}
    // first granule of group c (c = groups gives G): floor(c * G / n) = c * q + floor(c * r / n)
    __host__ __device__ int start(int c) const { return c * q + c * r / groups; }
    // the group that holds granule g: the last one whose range starts at or before g
    __host__ __device__ int group_of(int g) const
    {
        int c = (int)((float)g * (float)groups / (float)gtot);   // within one or two of the answer
        c = c < 0 ? 0 : c >= groups ? groups - 1 : c;
        while (c > 0 && start(c) > g) --c;
        while (c + 1 < groups && start(c + 1) <= g) ++c;
        return c;
    }
    // how many groups share the tile whose granules are [first, first + gpt)
    __host__ __device__ int groups_of_tile(int first, int gpt) const { return group_of(first + gpt - 1) - group_of(first) + 1; }
};

struct SlabSumArgs {
    const float *slabs;        // problem p, slab k: slabs + (p * KS + k) * slab, rows ld apart
    long long slab;
    float *O;
    long long ldo, stride_O;
    int ld, KS;
    int M, N, batch, Mt, Nt, NT;
    int gpt, bal_ctas;         // balanced partition: granules per row tile and CTAs (a tile's slab count follows); 0: KS slabs everywhere
    const int *flags;          // flags[0] | flags[1] != 0: the tile kernel did not run (the row kernels take over): nothing to add
};

__global__ void __launch_bounds__(256) slab_sum_kernel(const SlabSumArgs a)
{
    // The flags are final before the tile kernel lets its dependents start.  They are read BEFORE this grid lets its
    // own dependent go: that is the gated row kernel, whose last CTA clears flags[1] for the next call.
    const bool skip = (*reinterpret_cast<const volatile int *>(a.flags) | *reinterpret_cast<const volatile int *>(a.flags + 1)) != 0;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (skip) return;
    bool waited = false;   // (a thread works out where its first element is before it waits for the tile kernel)
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x, nthreads = (long long)gridDim.x * blockDim.x;
    const int n4 = (a.N + 3) >> 2;
    const long long total = (long long)a.batch * a.M * n4;
    const bool vec_out = (a.ldo & 3) == 0 && (a.stride_O & 3) == 0 && (reinterpret_cast<uintptr_t>(a.O) & 15) == 0;
    const bool small = total < 0x7fffffffll;   // 32-bit index arithmetic (64-bit divisions are library calls)
    const Balance balance(a.bal_ctas ? a.batch * a.Mt * a.gpt : 1, a.bal_ctas ? a.bal_ctas / a.Nt : 1);
    for (long long e = tid; e < total; e += nthreads) {
        int n, r, p;
        if (small) {
            const unsigned e32 = (unsigned)e, pr = e32 / (unsigned)n4;
            n = (int)(e32 - pr * (unsigned)n4) * 4;
            p = a.batch == 1 ? 0 : (int)(pr / (unsigned)a.M);
            r = (int)(pr - (unsigned)p * (unsigned)a.M);
        } else {
            n = (int)(e % n4) * 4;
            const long long pr = e / n4;
            r = (int)(pr % a.M);
            p = (int)(pr / a.M);
        }
        int cnt = a.KS;
        if (a.bal_ctas) cnt = balance.groups_of_tile((p * a.Mt + r / kSlabTileRows) * a.gpt, a.gpt);
        const float *src = a.slabs + (long long)p * a.KS * a.slab + (long long)r * a.ld + n;
        if (!waited) {
            asm volatile("griddepcontrol.wait;" ::: "memory");   // the tile kernel has completed: the slabs are whole
            waited = true;
        }
        // (the first four slabs' loads in flight together)
        float4 v[4];
#pragma unroll
        for (int k = 0; k < 4; ++k)
            if (k < cnt) v[k] = __ldcg(reinterpret_cast<const float4 *>(src + (long long)k * a.slab));
        float4 acc = v[0];
#pragma unroll
        for (int k = 1; k < 4; ++k)
            if (k < cnt) { acc.x += v[k].x; acc.y += v[k].y; acc.z += v[k].z; acc.w += v[k].w; }
        for (int k = 4; k < cnt; ++k) {
            const float4 w = __ldcg(reinterpret_cast<const float4 *>(src + (long long)k * a.slab));
            acc.x += w.x; acc.y += w.y; acc.z += w.z; acc.w += w.w;
        }
        float *dst = a.O + p * a.stride_O + (long long)r * a.ldo + n;
        if (n + 3 < a.N && vec_out) {
            *reinterpret_cast<float4 *>(dst) = acc;
        } else {
            dst[0] = acc.x;
            if (n + 1 < a.N) dst[1] = acc.y;
            if (n + 2 < a.N) dst[2] = acc.z;
            if (n + 3 < a.N) dst[3] = acc.w;
        }
    }
}

}  // namespace b2sp
