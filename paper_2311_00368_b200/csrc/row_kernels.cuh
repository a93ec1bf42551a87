// CUDA-core "row" kernels for SPMM / SDDMM / FusedMM over CSR (sm_100a).
//
// One CTA of kRowWarps warps owns one sparse row (and one slab of output columns).  The row's
// (col_idx, values) segment is consumed in chunks of 32 entries -- the paper's VLC = 32 -- one
// entry per lane, loaded coalesced and handed round by warp shuffles.  The warps of the CTA
// take alternate chunks (the paper's "NT threads share a row's nonzeros") and, for SPMM and
// FusedMM, their partial output rows are combined through shared memory in a fixed order, so
// results are deterministic.  Rows are visited in the order given by `row_order` (longest
// first, produced by the binning kernels below) or in natural order when it is NULL.
// `clear`, when not NULL, points at the workspace's status word, which the kernel resets (a call whose only
// launch is this kernel cannot fail on the device).
// `gate`, when not NULL, points at three device words (used when the row family is only the fallback of
// the dense-tile family): the kernel does nothing if words 0 and 1 are both 0.  Word 0 says that the
// window table cannot be used and stays as it is; word 1 says that a dense operand of this call holds a
// non-finite value and is per call: the last CTA of this grid to have read it clears it (word 2 counts
// the readers), so that the next call on the workspace starts clean without a launch of its own.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace b2sp {

constexpr int kRowWarps = 4;
constexpr int kRowThreads = kRowWarps * 32;
constexpr int kBuckets = 32;
constexpr unsigned kFull = 0xffffffffu;

// ------------------------------------------------------------------------------------------
// Row binning (work assignment): counting sort of the rows by length bucket
// bucket(len) = number of significant bits of len, longest bucket first.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ int bucket_of(int len) { return len <= 0 ? 0 : 32 - __clz(len); }

// Programmatic dependent launches: the binning kernels and the row kernel that follows them are chained so
// that each is placed, and does what does not need its predecessor's output, while the predecessor runs.
__device__ __forceinline__ void grid_release_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_wait_for_primary() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// A batch of independent problems of the same sizes in one launch (FusedMM only): blockIdx.z is the problem,
// whose arrays start `*` elements after those of problem 0.  All zero for a single problem.
struct RowBatch {
    long long rp, nz, A, B, D, O;
};
struct NoBatch {};   // what a single-problem kernel takes in RowBatch's place (no parameter bytes, no arithmetic)
template <bool BATCHED> struct BatchArg { using type = NoBatch; };
template <> struct BatchArg<true> { using type = RowBatch; };

// True when a gated launch has nothing to do (see the top of this file).  Called by every thread of the CTA.
__device__ __forceinline__ bool gate_closed(int *gate)
{
    if (!gate) return false;
    __shared__ int gate_word;
    if (threadIdx.x == 0) {
        volatile int *g = gate;
        gate_word = g[0] | g[1];
        __threadfence();   // the read above is performed before this CTA is counted as a reader
        const unsigned readers = gridDim.x * gridDim.y * gridDim.z;
        if ((unsigned)atomicAdd(gate + 2, 1) == readers - 1) {
            g[2] = 0;
            g[1] = 0;
        }
    }
    __syncthreads();
    return gate_word == 0;
}

__global__ void bin_count_kernel(int M, const int *__restrict__ row_ptr, int *__restrict__ count)
{
    __shared__ int h[kBuckets];
    grid_release_dependents();
    if (threadIdx.x < kBuckets) h[threadIdx.x] = 0;
    __syncthreads();
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < M) atomicAdd(&h[bucket_of(row_ptr[i + 1] - row_ptr[i])], 1);
    __syncthreads();
    if (threadIdx.x < kBuckets && h[threadIdx.x]) atomicAdd(&count[threadIdx.x], h[threadIdx.x]);
}

__global__ void bin_scatter_kernel(int M, const int *__restrict__ row_ptr,
                                   const int *__restrict__ count, int *__restrict__ cursor,
                                   int *__restrict__ row_order)
{
    __shared__ int h[kBuckets];
    __shared__ int base[kBuckets];
    if (threadIdx.x < kBuckets) h[threadIdx.x] = 0;
    __syncthreads();
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    int b = 0, r = 0;
    if (i < M) {
        b = bucket_of(row_ptr[i + 1] - row_ptr[i]);
        r = atomicAdd(&h[b], 1);
    }
    __syncthreads();
    grid_wait_for_primary();     // the counts of the whole matrix (bin_count_kernel)
    grid_release_dependents();   // the row kernel behind this one waits for this grid before it reads the order
    if (threadIdx.x < kBuckets) {
        int mine = threadIdx.x, start = 0;
        for (int j = kBuckets - 1; j > mine; --j) start += count[j];
        base[mine] = h[mine] ? start + atomicAdd(&cursor[mine], h[mine]) : 0;
    }
    __syncthreads();
    if (i < M) row_order[base[b] + r] = i;
}

// ------------------------------------------------------------------------------------------
// helpers
// ------------------------------------------------------------------------------------------
// Dense operands are fp32 or bfloat16 (DT below); sums and outputs are always fp32.  A bf16 value is the top
// half of the fp32 value it stands for, so widening it is exact.
struct bf16_t { unsigned short bits; };
__device__ __forceinline__ float4 ldg4(const float *p) { return __ldg(reinterpret_cast<const float4 *>(p)); }
__device__ __forceinline__ float4 ldg4(const bf16_t *p)   // four consecutive elements, 8-byte aligned
{
    const uint2 u = __ldg(reinterpret_cast<const uint2 *>(p));
    return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u),
                       __uint_as_float(u.y << 16), __uint_as_float(u.y & 0xffff0000u));
}
__device__ __forceinline__ float ldg1(const float *p) { return __ldg(p); }
__device__ __forceinline__ float ldg1(const bf16_t *p)
{
    return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short *>(p)) << 16);
}

__device__ __forceinline__ void fma4(float4 &acc, float s, const float4 &v)
{
    acc.x = fmaf(s, v.x, acc.x);
    acc.y = fmaf(s, v.y, acc.y);
    acc.z = fmaf(s, v.z, acc.z);
    acc.w = fmaf(s, v.w, acc.w);
}

__device__ __forceinline__ float dot4(const float4 &a, const float4 &b, float acc)
{
    acc = fmaf(a.x, b.x, acc);
    acc = fmaf(a.y, b.y, acc);
    acc = fmaf(a.z, b.z, acc);
    acc = fmaf(a.w, b.w, acc);
    return acc;
}

// Geometry of the SPMM sweep.  SPLIT sub-warps of LPN = 32/SPLIT lanes each take alternate
// entries of a chunk; a lane owns U float4 column groups: columns col0 + (sl + LPN*u)*4.
template <int U, int SPLIT>
struct SweepGeom {
    static constexpr int LPN = 32 / SPLIT;
    static constexpr int SLAB = LPN * 4 * U;
};

// One chunk (up to 32 entries, lane l holds entry l: column k, scalar s) of the Alg. 2 SAXPY
// sweep.  SRC(j) gives the lane that holds entry j's scalar.
template <int U, int SPLIT, bool PERMUTED, typename DT>
__device__ __forceinline__ void saxpy_chunk(float4 (&acc)[U], int k, float s, int cnt,
                                            const DT *__restrict__ Dcol, int64_t ldd,
                                            bool (&live)[U], int sub)
{
    constexpr int LPN = 32 / SPLIT;
    constexpr int STEPS = 32 / SPLIT;
    if (cnt == 32) {
#pragma unroll 8
        for (int jj = 0; jj < STEPS; ++jj) {
            int j = jj * SPLIT + sub;
            int src = PERMUTED ? ((j & 3) * 8 + (j >> 2)) : j;
            int kk = __shfl_sync(kFull, k, j);
            float ss = __shfl_sync(kFull, s, src);
            const DT *d = Dcol + (int64_t)kk * ldd;
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (live[u]) fma4(acc[u], ss, ldg4(d + u * LPN * 4));
        }
    } else {
        for (int jj = 0; jj < STEPS; ++jj) {
            int j = jj * SPLIT + sub;
            int src = PERMUTED ? ((j & 3) * 8 + (j >> 2)) : j;
            int kk = __shfl_sync(kFull, k, j);
            float ss = __shfl_sync(kFull, s, src);
            if (j < cnt) {
                const DT *d = Dcol + (int64_t)kk * ldd;
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (live[u]) fma4(acc[u], ss, ldg4(d + u * LPN * 4));
            }
        }
    }
}

// Combine the sub-warps of a warp, then the warps of the CTA (fixed order), and store the row.
template <int U, int SPLIT>
__device__ __forceinline__ void reduce_and_store_row(float4 (&acc)[U], float4 *red, int warp,
                                                     int lane, float *__restrict__ Orow,
                                                     bool (&live)[U])
{
    constexpr int LPN = 32 / SPLIT;
#pragma unroll
    for (int off = 16; off >= LPN; off >>= 1) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            acc[u].x += __shfl_xor_sync(kFull, acc[u].x, off);
            acc[u].y += __shfl_xor_sync(kFull, acc[u].y, off);
            acc[u].z += __shfl_xor_sync(kFull, acc[u].z, off);
            acc[u].w += __shfl_xor_sync(kFull, acc[u].w, off);
        }
    }
    if (lane < LPN) {
#pragma unroll
        for (int u = 0; u < U; ++u) red[(warp * U + u) * LPN + lane] = acc[u];
    }
    __syncthreads();
    if (warp == 0 && lane < LPN) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (!live[u]) continue;
            float4 r = red[u * LPN + lane];
#pragma unroll
            for (int w = 1; w < kRowWarps; ++w) {
                float4 t = red[(w * U + u) * LPN + lane];
                r.x += t.x; r.y += t.y; r.z += t.z; r.w += t.w;
            }
            *reinterpret_cast<float4 *>(Orow + u * LPN * 4) = r;
        }
    }
}

// ------------------------------------------------------------------------------------------
// SPMM  (Alg. 2; float4 path: N, ldd, ldo multiples of 4, D and O 16-byte aligned)
// ------------------------------------------------------------------------------------------
template <int U, int SPLIT, typename DT>
__global__ void __launch_bounds__(kRowThreads)
spmm_row_kernel(int N, const int *__restrict__ row_ptr, const int *__restrict__ col_idx,
                const float *__restrict__ values, const DT *__restrict__ D, int64_t ldd,
                float *__restrict__ O, int64_t ldo, const int *__restrict__ row_order,
                int *__restrict__ gate, int nrows, int *__restrict__ clear)
{
    using G = SweepGeom<U, SPLIT>;
    __shared__ float4 red[kRowWarps * U * G::LPN];
    if (gate_closed(gate)) return;
    if (clear && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) *clear = 0;
    if (row_order) grid_wait_for_primary();   // launched behind the binning pass: its row order
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane / G::LPN, sl = lane % G::LPN;
    for (int rb = blockIdx.x; rb < nrows; rb += gridDim.x) {
        const int row = row_order ? row_order[rb] : rb;
        const int col0 = blockIdx.y * G::SLAB + sl * 4;
        bool live[U];
        float4 acc[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            live[u] = col0 + u * G::LPN * 4 < N;
            acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        const int beg = row_ptr[row], end = row_ptr[row + 1];
        const DT *Dcol = D + col0;
        // the next chunk's indices and values are fetched before the current chunk is consumed
        // (the role of the paper's prefetch of the next ja/avalues block)
        int k = 0;
        float s = 0.f;
        {
            int p = beg + warp * 32 + lane;
            if (p < end) {
                k = __ldg(col_idx + p);
                s = __ldg(values + p);
            }
        }
        for (int c = beg + warp * 32; c < end; c += kRowWarps * 32) {
            int pn = c + kRowWarps * 32 + lane;
            int kn = 0;
            float sn = 0.f;
            if (pn < end) {
                kn = __ldg(col_idx + pn);
                sn = __ldg(values + pn);
            }
            saxpy_chunk<U, SPLIT, false, DT>(acc, k, s, min(32, end - c), Dcol, ldd, live, sub);
            k = kn;
            s = sn;
        }
        reduce_and_store_row<U, SPLIT>(acc, red, warp, lane, O + (int64_t)row * ldo + col0, live);
        __syncthreads();   // shared memory is reused by the next row
    }
}

// Scalar path for any N / ld / alignment: a lane owns columns col0 + lane + 32u (u < 4).
template <typename DT>
__global__ void __launch_bounds__(kRowThreads)
spmm_row_scalar_kernel(int N, const int *__restrict__ row_ptr, const int *__restrict__ col_idx,
                       const float *__restrict__ values, const DT *__restrict__ D, int64_t ldd,
                       float *__restrict__ O, int64_t ldo, const int *__restrict__ row_order,
                       int *__restrict__ gate, int nrows, int *__restrict__ clear)
{
    __shared__ float red[kRowWarps][128];
    if (gate_closed(gate)) return;
    if (clear && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) *clear = 0;
    if (row_order) grid_wait_for_primary();   // launched behind the binning pass: its row order
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int rb = blockIdx.x; rb < nrows; rb += gridDim.x) {
        const int row = row_order ? row_order[rb] : rb;
        const int col0 = blockIdx.y * 128 + lane;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        const int beg = row_ptr[row], end = row_ptr[row + 1];
        for (int c = beg + warp * 32; c < end; c += kRowWarps * 32) {
            int p = c + lane;
            int k = 0;
            float s = 0.f;
            if (p < end) {
                k = __ldg(col_idx + p);
                s = __ldg(values + p);
            }
            int cnt = min(32, end - c);
            for (int j = 0; j < cnt; ++j) {
                int kk = __shfl_sync(kFull, k, j);
                float ss = __shfl_sync(kFull, s, j);
                const DT *d = D + (int64_t)kk * ldd + col0;
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (col0 + 32 * u < N) acc[u] = fmaf(ss, ldg1(d + 32 * u), acc[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) red[warp][lane + 32 * u] = acc[u];
        __syncthreads();
        if (warp == 0) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (col0 + 32 * u >= N) continue;
                float r = red[0][lane + 32 * u];
                for (int w = 1; w < kRowWarps; ++w) r += red[w][lane + 32 * u];
                O[(int64_t)row * ldo + col0 + 32 * u] = r;
            }
        }
        __syncthreads();   // shared memory is reused by the next row
    }
}

// ------------------------------------------------------------------------------------------
// SDDMM  (Alg. 1; float4 path: Kd, lda, ldb multiples of 4, A and B 16-byte aligned)
//
// A group of 8 lanes computes one sampled dot product: lane t of the group owns elements
// (t + 8u)*4 .. +3 of the Kd-vector.  KU > 0: A_i is held in KU float4 registers per lane
// (Kd <= 32*KU).  KU == 0: any Kd, A_i staged in shared memory.  In a chunk of 32 entries,
// group g takes entries 4r + g (r = 0..7); after the 3-step butterfly every lane of the
// group has the sum and lane t keeps round t's, so lane 8g + t ends up holding entry 4t + g.
// ------------------------------------------------------------------------------------------
template <int KU, typename DT>
__device__ __forceinline__ float sddmm_chunk(const float4 (&areg)[KU > 0 ? KU : 1],
                                             const float *__restrict__ a_smem, int Kd, int k,
                                             const DT *__restrict__ B, int64_t ldb, int lane)
{
    const int g = lane >> 3, t = lane & 7;
    float mine = 0.f;
#pragma unroll 4
    for (int r = 0; r < 8; ++r) {
        int kq = __shfl_sync(kFull, k, 4 * r + g);
        const DT *b = B + (int64_t)kq * ldb + t * 4;
        float part = 0.f;
        if (KU > 0) {
#pragma unroll
            for (int u = 0; u < KU; ++u)
                if ((t + 8 * u) * 4 < Kd) part = dot4(areg[u], ldg4(b + u * 32), part);
        } else {
            for (int e = t * 4; e < Kd; e += 32)
                part = dot4(*reinterpret_cast<const float4 *>(a_smem + e), ldg4(b + e - t * 4), part);
        }
        part += __shfl_xor_sync(kFull, part, 1);
        part += __shfl_xor_sync(kFull, part, 2);
        part += __shfl_xor_sync(kFull, part, 4);
        if (r == t) mine = part;
    }
    return mine;  // lane 8g+t: dot product of entry 4t+g
}

template <int KU, typename DT>
__device__ __forceinline__ void load_a_row(float4 (&areg)[KU > 0 ? KU : 1], float *a_smem,
                                           const DT *__restrict__ Arow, int Kd, int lane)
{
    if (KU > 0) {
        const int t = lane & 7;
#pragma unroll
        for (int u = 0; u < (KU > 0 ? KU : 1); ++u)
            areg[u] = (t + 8 * u) * 4 < Kd ? ldg4(Arow + (t + 8 * u) * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
    } else {
        for (int e = threadIdx.x * 4; e < Kd; e += kRowThreads * 4)
            *reinterpret_cast<float4 *>(a_smem + e) = ldg4(Arow + e);
        __syncthreads();
    }
}

template <int KU, typename DT>
__global__ void __launch_bounds__(kRowThreads)
sddmm_row_kernel(int Kd, const int *__restrict__ row_ptr, const int *__restrict__ col_idx,
                 const float *s_values, const DT *__restrict__ A, int64_t lda,
                 const DT *__restrict__ B, int64_t ldb, float *out_values,
                 const int *__restrict__ row_order, int *__restrict__ gate, int nrows, int *__restrict__ clear)
{
    extern __shared__ float4 dyn_smem[];
    float *a_smem = reinterpret_cast<float *>(dyn_smem);
    if (gate_closed(gate)) return;
    if (clear && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) *clear = 0;
    if (row_order) grid_wait_for_primary();   // launched behind the binning pass: its row order
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int rb = blockIdx.x; rb < nrows; rb += gridDim.x) {
        const int row = row_order ? row_order[rb] : rb;
        const int beg = row_ptr[row], end = row_ptr[row + 1];
        float4 areg[KU > 0 ? KU : 1];
        load_a_row<KU, DT>(areg, a_smem, A + (int64_t)row * lda, Kd, lane);
        const int slot = (lane & 7) * 4 + (lane >> 3);  // entry of the chunk this lane ends up holding
        for (int c = beg + warp * 32; c < end; c += kRowWarps * 32) {
            int p = c + lane;
            int k = p < end ? __ldg(col_idx + p) : 0;
            float dp = sddmm_chunk<KU, DT>(areg, a_smem, Kd, k, B, ldb, lane);
            int q = c + slot;
            if (q < end) out_values[q] = s_values ? s_values[q] * dp : dp;
        }
        __syncthreads();   // shared memory is reused by the next row
    }
}

// Scalar path for any Kd / ld / alignment: one lane per entry, serial dot product.
template <typename DT>
__global__ void __launch_bounds__(kRowThreads)
sddmm_row_scalar_kernel(int Kd, const int *__restrict__ row_ptr, const int *__restrict__ col_idx,
                        const float *s_values, const DT *__restrict__ A, int64_t lda,
                        const DT *__restrict__ B, int64_t ldb, float *out_values,
                        const int *__restrict__ row_order, int *__restrict__ gate, int nrows, int *__restrict__ clear)
{
    if (gate_closed(gate)) return;
    if (clear && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) *clear = 0;
    if (row_order) grid_wait_for_primary();   // launched behind the binning pass: its row order
    for (int rb = blockIdx.x; rb < nrows; rb += gridDim.x) {
        const int row = row_order ? row_order[rb] : rb;
        const int beg = row_ptr[row], end = row_ptr[row + 1];
        const DT *a = A + (int64_t)row * lda;
        for (int p = beg + threadIdx.x; p < end; p += kRowThreads) {
            const DT *b = B + (int64_t)__ldg(col_idx + p) * ldb;
            float dp = 0.f;
            for (int l = 0; l < Kd; ++l) dp = fmaf(ldg1(a + l), ldg1(b + l), dp);
            out_values[p] = s_values ? s_values[p] * dp : dp;
        }
        __syncthreads();   // shared memory is reused by the next row
    }
}

// ------------------------------------------------------------------------------------------
// FusedMM  (Alg. 3): per chunk, the SDDMM values stay in registers (one per lane) and are the
// scalars of the SAXPY sweep over the same staged column indices; C never reaches memory.
// ------------------------------------------------------------------------------------------
template <int KU, int U, int SPLIT, bool BATCHED, typename DT>
__global__ void __launch_bounds__(kRowThreads)
fusedmm_row_kernel(int Kd, int N, const int *__restrict__ row_ptr, const int *__restrict__ col_idx,
                   const float *__restrict__ s_values, const DT *__restrict__ A, int64_t lda,
                   const DT *__restrict__ B, int64_t ldb, const DT *__restrict__ D,
                   int64_t ldd, float *__restrict__ O, int64_t ldo,
                   const int *__restrict__ row_order, int *__restrict__ gate, int nrows, int *__restrict__ clear,
                   typename BatchArg<BATCHED>::type batch)
{
    using G = SweepGeom<U, SPLIT>;
    extern __shared__ float4 dyn_smem[];
    if (gate_closed(gate)) return;
    if constexpr (BATCHED) {   // this problem's arrays
        const long long pb = blockIdx.z;
        row_ptr += pb * batch.rp; col_idx += pb * batch.nz; if (s_values) s_values += pb * batch.nz;
        A += pb * batch.A; B += pb * batch.B; D += pb * batch.D; O += pb * batch.O;
    }
    if (clear && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) *clear = 0;
    if (row_order) grid_wait_for_primary();   // launched behind the binning pass: its row order
    float4 *red = dyn_smem;                                                   // kRowWarps*U*LPN
    float *a_smem = reinterpret_cast<float *>(dyn_smem + kRowWarps * U * G::LPN);  // Kd (KU == 0)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane / G::LPN, sl = lane % G::LPN;
    for (int rb = blockIdx.x; rb < nrows; rb += gridDim.x) {
        const int row = row_order ? row_order[rb] : rb;
        const int col0 = blockIdx.y * G::SLAB + sl * 4;
        bool live[U];
        float4 acc[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            live[u] = col0 + u * G::LPN * 4 < N;
            acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        const int beg = row_ptr[row], end = row_ptr[row + 1];
        float4 areg[KU > 0 ? KU : 1];
        load_a_row<KU, DT>(areg, a_smem, A + (int64_t)row * lda, Kd, lane);
        const int slot = (lane & 7) * 4 + (lane >> 3);
        const DT *Dcol = D + col0;
        int k = 0;
        float sv = 1.f;
        {
            int p = beg + warp * 32 + lane, q = beg + warp * 32 + slot;
            if (p < end) k = __ldg(col_idx + p);
            if (s_values && q < end) sv = __ldg(s_values + q);
        }
        for (int c = beg + warp * 32; c < end; c += kRowWarps * 32) {
            int pn = c + kRowWarps * 32 + lane, qn = c + kRowWarps * 32 + slot;
            int kn = pn < end ? __ldg(col_idx + pn) : 0;
            float svn = (s_values && qn < end) ? __ldg(s_values + qn) : 1.f;
            float cv = sv * sddmm_chunk<KU, DT>(areg, a_smem, Kd, k, B, ldb, lane);
            saxpy_chunk<U, SPLIT, true, DT>(acc, k, cv, min(32, end - c), Dcol, ldd, live, sub);
            k = kn;
            sv = svn;
        }
        reduce_and_store_row<U, SPLIT>(acc, red, warp, lane, O + (int64_t)row * ldo + col0, live);
        __syncthreads();   // shared memory is reused by the next row
    }
}

// Scalar path for any widths / alignment: lane-per-entry dot products, then a scalar sweep.
template <typename DT>
__global__ void __launch_bounds__(kRowThreads)
fusedmm_row_scalar_kernel(int Kd, int N, const int *__restrict__ row_ptr,
                          const int *__restrict__ col_idx, const float *__restrict__ s_values,
                          const DT *__restrict__ A, int64_t lda, const DT *__restrict__ B,
                          int64_t ldb, const DT *__restrict__ D, int64_t ldd,
                          float *__restrict__ O, int64_t ldo, const int *__restrict__ row_order,
                          int *__restrict__ gate, int nrows, int *__restrict__ clear, RowBatch batch)
{
    __shared__ float red[kRowWarps][128];
    if (gate_closed(gate)) return;
    {   // this problem's arrays
        const long long pb = blockIdx.z;
        row_ptr += pb * batch.rp; col_idx += pb * batch.nz; if (s_values) s_values += pb * batch.nz;
        A += pb * batch.A; B += pb * batch.B; D += pb * batch.D; O += pb * batch.O;
    }
    if (clear && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) *clear = 0;
    if (row_order) grid_wait_for_primary();   // launched behind the binning pass: its row order
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int rb = blockIdx.x; rb < nrows; rb += gridDim.x) {
        const int row = row_order ? row_order[rb] : rb;
        const int col0 = blockIdx.y * 128 + lane;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        const int beg = row_ptr[row], end = row_ptr[row + 1];
        const DT *a = A + (int64_t)row * lda;
        for (int c = beg + warp * 32; c < end; c += kRowWarps * 32) {
            int p = c + lane;
            int k = 0;
            float cv = 0.f;
            if (p < end) {
                k = __ldg(col_idx + p);
                const DT *b = B + (int64_t)k * ldb;
                for (int l = 0; l < Kd; ++l) cv = fmaf(ldg1(a + l), ldg1(b + l), cv);
                if (s_values) cv *= __ldg(s_values + p);
            }
            int cnt = min(32, end - c);
            for (int j = 0; j < cnt; ++j) {
                int kk = __shfl_sync(kFull, k, j);
                float ss = __shfl_sync(kFull, cv, j);
                const DT *d = D + (int64_t)kk * ldd + col0;
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (col0 + 32 * u < N) acc[u] = fmaf(ss, ldg1(d + 32 * u), acc[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) red[warp][lane + 32 * u] = acc[u];
        __syncthreads();
        if (warp == 0) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (col0 + 32 * u >= N) continue;
                float r = red[0][lane + 32 * u];
                for (int w = 1; w < kRowWarps; ++w) r += red[w][lane + 32 * u];
                O[(int64_t)row * ldo + col0 + 32 * u] = r;
            }
        }
        __syncthreads();   // shared memory is reused by the next row
    }
}

// ------------------------------------------------------------------------------------------
// CSR validation (debug helper)
// ------------------------------------------------------------------------------------------
__global__ void validate_csr_kernel(int M, int K, long long nnz, const int *__restrict__ row_ptr,
                                    const int *__restrict__ col_idx, int *__restrict__ flag)
{
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    long long stride = (long long)gridDim.x * blockDim.x;
    bool bad = false;
    if (i == 0) bad |= row_ptr[0] != 0 || (long long)row_ptr[M] != nnz;
    for (long long r = i; r < M; r += stride) bad |= row_ptr[r + 1] < row_ptr[r];
    for (long long p = i; p < nnz; p += stride) {
        int c = col_idx[p];
        bad |= c < 0 || c >= K;
    }
    if (bad) atomicExch(flag, 1);
}

}  // namespace b2sp
