// Support kernels of the dense-tile (tensor-core) family.
//
// Idea of the family: at 10-30% density a 128 x 32 window of S is a dense tile with 70-90% zeros, and
// the 5th-generation tensor cores multiply it by a dense tile an order of magnitude faster than the
// FP32 pipes can walk its nonzeros.  fp32 accuracy is kept by splitting every operand into two tf32
// numbers (x = hi + lo) and issuing three MMAs per product: hi*hi + lo*hi + hi*lo.
//
// Pieces here (the tile kernel itself is in tile_fused.cuh):
//   tile_masks_kernel      per row and 32-column window: first CSR position + occupancy bit mask
//                          (needs strictly increasing columns in a row; sets a flag otherwise)
//   split_dense_kernel     dense fp32 operands -> zero-padded (hi, lo) tf32 copies
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx_sm100.cuh"
#include "tile_dispatch.h"

namespace b2sp {

constexpr int kTileKC = 32;       // columns of S per pipeline stage (one 128-byte swizzle row of tf32)
// Flag words of the tile pre-passes (the gate of the row-kernel fallback reads the first two, see row_kernels.cuh):
constexpr int kFlagUnsorted = 0;   // != 0: the window table is unusable (a row's columns are not strictly increasing,
                                   // or the table belongs to other arrays); stays set until the table is rebuilt
constexpr int kFlagNotFinite = 1;  // != 0: a dense operand of this call holds a non-finite value; cleared by the fallback
constexpr int kFlagGateReaders = 2;  // CTAs of the gated fallback that have read the flags so far

// ---- table signature ------------------------------------------------------------------------------------
struct PatternSignature {
    int magic, M, K, Wk;
    long long nnz;
    const int *row_ptr, *col_idx;
    long long batch, rp_stride, nz_stride;   // a batch of patterns (see tile_masks_kernel); 1, 0, 0 for a single one
};
constexpr int kPatternMagic = 0x62327370;

// ---- window table -------------------------------------------------------------------------------
// T[r*Wk + w] = (first CSR position of row r whose column is >= 32w, occupancy bit mask of the column
// window [32w, 32w+32): bit b set <=> column 32w+b is stored).
// One block of four warps per row (rows differ a lot in length; blocks are scheduled as they finish),
// one mask word per window of the row in shared memory.  First sweep: the warps read the row's column
// indices 128 at a time (coalesced, four per lane); a lane merges the bits of its entries that fall
// into the same window and ORs them into the window's word (shared-memory atomics).  Second sweep: thread = window; the
// position of a window is the row start plus the entries of all earlier windows (a block prefix sum
// over the pop counts).  Every window of every row is written, so the table needs no clearing.
// The table is only meaningful when the columns of each row are strictly increasing and in range;
// the first sweep checks exactly that and sets flags[kFlagUnsorted] if not.
constexpr int kMasksWarps = 4;
constexpr int kMasksMaxWk = 24 * 1024;   // the mask row must fit in the shared memory a block may ask for (96 KB)

// A batch of `sig.batch` patterns of the same M and K (row_ptr arrays `sig.rp_stride` elements apart, each
// starting at 0; col_idx arrays `sig.nz_stride` elements apart) gives one table per pattern, stacked:
// T[(b*M + r)*Wk + w], positions relative to the pattern's own col_idx array.
__global__ void __launch_bounds__(kMasksWarps * 32)
tile_masks_kernel(int M, int K, int Wk, long long nnz, const int *__restrict__ row_ptr0,
                  const int *__restrict__ col_idx0, int2 *__restrict__ T, int *__restrict__ flags,
                  PatternSignature sig, PatternSignature *__restrict__ sig_out)
{
    extern __shared__ __align__(16) unsigned mask[];     // Wk words
    // (inside a stateless tile op the operand-split kernel is launched as a programmatic dependent of this
    // one: the two touch different data and may overlap; that kernel waits for this grid before it ends)
    ptx::launch_dependents();
    if (blockIdx.x == 0 && threadIdx.x == 0) *sig_out = sig;   // what the table is built from
    __shared__ int warp_total[kMasksWarps];
    constexpr unsigned kFull = 0xffffffffu;
    constexpr int NT = kMasksWarps * 32;
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    bool bad = false;
    const long long rows_all = (long long)M * sig.batch;
    for (long long rowg = blockIdx.x; rowg < rows_all; rowg += gridDim.x) {
        const int pb = sig.batch == 1 ? 0 : (int)(rowg / M), row = (int)(rowg - (long long)pb * M);   // (no 64-bit division for a single pattern)
        const int *__restrict__ row_ptr = row_ptr0 + pb * sig.rp_stride;
        const int *__restrict__ col_idx = col_idx0 + pb * sig.nz_stride;
        const bool vec = (reinterpret_cast<uintptr_t>(col_idx) & 15) == 0;
        for (int w = threadIdx.x; w < Wk; w += NT) mask[w] = 0u;
        __syncthreads();
        const int beg = __ldg(row_ptr + row), end = __ldg(row_ptr + row + 1);
        // lane l of a warp takes positions p .. p + 3 (one 16-byte load when the array allows it); the
        // warp's next load is in flight while this one is checked.
        auto load4 = [&](int p) {
            int4 c = make_int4(0, 0, 0, 0);
            if (p >= end) return c;
            if (vec && p + 3 < nnz) return __ldg(reinterpret_cast<const int4 *>(col_idx + p));
            c.x = __ldg(col_idx + p);
            if (p + 1 < end) c.y = __ldg(col_idx + p + 1);
            if (p + 2 < end) c.z = __ldg(col_idx + p + 2);
            if (p + 3 < end) c.w = __ldg(col_idx + p + 3);
            return c;
        };
        const int abeg = beg & ~3;
        int4 c_next = load4(abeg + 128 * wib + 4 * lane);
        for (int p0 = abeg + 128 * wib; p0 < end; p0 += 128 * kMasksWarps) {
            const int p = p0 + 4 * lane;
            const int4 c = c_next;
            c_next = load4(p + 128 * kMasksWarps);
            int prev = __shfl_up_sync(kFull, c.w, 1);
            if (lane == 0 && p > beg) prev = __ldg(col_idx + p - 1);
            const bool inside = p >= beg && p + 3 < end;
            const bool in_range = (unsigned)c.x < (unsigned)K && (unsigned)c.y < (unsigned)K &&
                                  (unsigned)c.z < (unsigned)K && (unsigned)c.w < (unsigned)K;
            if (inside && in_range) {
                // common case: four valid entries, almost always in one or two windows
                bad |= (p > beg && c.x <= prev) || c.y <= c.x || c.z <= c.y || c.w <= c.z;
                const int wx = c.x >> 5, wy = c.y >> 5, wz = c.z >> 5, ww = c.w >> 5;
                const unsigned bx = 1u << (c.x & 31), by = 1u << (c.y & 31), bz = 1u << (c.z & 31), bw = 1u << (c.w & 31);
                atomicOr(&mask[wx], bx | (wy == wx ? by : 0u) | (wz == wx ? bz : 0u) | (ww == wx ? bw : 0u));
                if (ww != wx) {
                    atomicOr(&mask[ww], bw | (wz == ww ? bz : 0u) | (wy == ww ? by : 0u));
                    if (wy != wx && wy != ww) atomicOr(&mask[wy], by);
                    if (wz != wx && wz != ww) atomicOr(&mask[wz], bz);
                }
            } else {
                auto visit = [&](int q, int col, int before) {
                    if (q >= beg && q < end) {
                        const bool ok = (unsigned)col < (unsigned)K;
                        bad |= !ok || (q > beg && col <= before);
                        if (ok) atomicOr(&mask[col >> 5], 1u << (col & 31));
                    }
                };
                visit(p, c.x, prev);
                visit(p + 1, c.y, c.x);
                visit(p + 2, c.z, c.y);
                visit(p + 3, c.w, c.z);
            }
        }
        __syncthreads();
        int run = beg;
        for (int w0 = 0; w0 < Wk; w0 += NT) {
            const int w = w0 + threadIdx.x;
            const unsigned m = w < Wk ? mask[w] : 0u;
            const int cnt = __popc(m);
            int incl = cnt;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int t = __shfl_up_sync(kFull, incl, d);
                if (lane >= d) incl += t;
            }
            if (lane == 31) warp_total[wib] = incl;
            __syncthreads();
            int before = 0, all = 0;
#pragma unroll
            for (int i = 0; i < kMasksWarps; ++i) {
                const int t = warp_total[i];
                if (i < wib) before += t;
                all += t;
            }
            if (w < Wk) T[(size_t)rowg * Wk + w] = make_int2(run + before + incl - cnt, (int)m);
            run += all;
            __syncthreads();   // warp_total and mask are reused
        }
    }
    if (bad) atomicExch(&flags[kFlagUnsorted], 1);
}

// True when the workspace holds a table built from exactly these arrays.
__device__ __forceinline__ bool signature_matches(const PatternSignature &want, const PatternSignature *have)
{
    const PatternSignature h = *have;
    return h.magic == want.magic && h.M == want.M && h.K == want.K && h.Wk == want.Wk && h.nnz == want.nnz &&
           h.row_ptr == want.row_ptr && h.col_idx == want.col_idx && h.batch == want.batch &&
           h.rp_stride == want.rp_stride && h.nz_stride == want.nz_stride;
}

// ---- dense operand split ----------------------------------------------------------------------------
// X [rows x cols] (ld) -> hi, lo in a column-blocked layout: element (r, c) lives at
// ((c/32)*rows_p + r)*32 + c%32, i.e. [cols_p/32][rows_p][32] floats, zero in the padding
// (rows_p >= rows, cols_p >= cols, cols_p % 32 == 0).  One 32-float group of a row is one
// 128-byte swizzle row for TMA, and the whole thing is a plain packed 3-D tensor.
// A batch of `batch` equally sized operands, `batch_stride` elements apart, is stacked along the rows:
// [cols_p/32][batch * rows_p][32].
// bf16 operands (dtype 1) are exact in tf32: hi is the value itself and no lo copy is written.
// One launch handles up to three jobs (blockIdx.y picks the job) and, being the first kernel of
// every tile op, also clears the workspace's device status word (unless `status` is NULL: the second
// kernel of a two-phase op keeps what the first one reported).
//
// The dense-tile kernels multiply whole windows of S, positions without a stored entry included (by
// zero), so an Inf or NaN anywhere in a dense operand -- also in a row no stored entry refers to -- or a
// value so close to FLT_MAX that its tf32 hi part rounds to Inf would turn into NaN in outputs that
// Eq. 1-3 leave finite.  Every job therefore also looks at what it reads, and a job with `check_only`
// (the A operand, which the tile kernel splits itself) does nothing else: a non-finite hi part raises
// the fallback flag, and the row kernels, which touch exactly the entries the equations name, produce
// the result.
struct SplitJob {
    const void *X;
    long long ld;
    int rows, cols;
    float *hi, *lo;
    int rows_p, cols_p;
    int batch;                // operands stacked along the rows (1: a single operand)
    long long batch_stride;   // elements between consecutive operands of the batch
    int dtype;                // kDenseF32 / kDenseBf16
    int check_only;           // look for non-finite values, write nothing
};


// It also compares the signature stored beside a prepared window table with the arrays of this call
// (`chk.have` != NULL) and raises the fallback flag on a mismatch: the flags are then final before the tile
// kernel starts, which lets the gated fallback run beside it.
struct TableCheck {
    PatternSignature want;
    const PatternSignature *have;   // NULL: nothing to check (the table was built by this call)
    int *flags;
    int after_prepass;              // launched as a programmatic dependent of the pattern pre-pass of the same call:
                                    // this grid must not complete before that one (the tile kernel waits for this grid only)
};

struct SplitJobs {
    SplitJob j[2];    // operands to split (blockIdx.y picks one)
    int n;
    SplitJob check;   // a check_only job done on the side by the blocks of job 0 (no blocks of its own: the launch
    int has_check;    // stays one wave of blocks, and the tile kernel behind it waits for this grid to end)
};

__device__ __forceinline__ bool tf32_hi_not_finite(uint32_t hi) { return (hi & 0x7f800000u) == 0x7f800000u; }

// One job of split_dense_kernel, walked by the blocks (gridDim.x of them) of one blockIdx.y.  True: a non-finite hi part was seen.
__device__ __forceinline__ bool split_job(const SplitJob &j)
{
    const bool bf16 = j.dtype == kDenseBf16;
    // 16-byte loads of four fp32 (or 8-byte loads of four bf16) need the alignment for every operand of the batch
    const bool vec = (j.ld & 3) == 0 && (j.batch_stride & 3) == 0 &&
                     (reinterpret_cast<uintptr_t>(j.X) & (bf16 ? 7 : 15)) == 0;
    const long long rows_all = (long long)j.batch * j.rows_p;
    const long long groups = rows_all * (j.cols_p >> 2);  // float4 groups
    const bool small = groups < 0x7fffffffll;
    bool bad = false;
    for (long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x; g < groups;
         g += (long long)gridDim.x * blockDim.x) {
        const int q = (int)(g & 7);                 // float4 inside the 32-float group
        const long long rg = g >> 3;                // (column group, stacked row) pair
        int b, r, c;
        if (small) {   // 32-bit index arithmetic (64-bit divisions are library calls: they were most of this kernel's time)
            const unsigned rg32 = (unsigned)rg, cg = rg32 / (unsigned)rows_all, rs = rg32 - cg * (unsigned)rows_all;
            b = j.batch == 1 ? 0 : (int)(rs / (unsigned)j.rows_p);
            r = (int)(rs - (unsigned)b * (unsigned)j.rows_p);
            c = (int)cg * 32 + q * 4;
        } else {
            const long long rs = rg % rows_all;
            b = (int)(rs / j.rows_p);
            r = (int)(rs % j.rows_p);
            c = (int)(rg / rows_all) * 32 + q * 4;
        }
        uint32_t h[4] = {0, 0, 0, 0}, l[4] = {0, 0, 0, 0};
        if (r < j.rows && c < j.cols) {
            const long long at = (long long)b * j.batch_stride + (long long)r * j.ld + c;
            float x[4] = {0.f, 0.f, 0.f, 0.f};
            if (bf16) {
                const unsigned short *src = static_cast<const unsigned short *>(j.X) + at;
                if (vec && c + 3 < j.cols) {
                    const uint2 u = __ldg(reinterpret_cast<const uint2 *>(src));
                    x[0] = __uint_as_float(u.x << 16); x[1] = __uint_as_float(u.x & 0xffff0000u);
                    x[2] = __uint_as_float(u.y << 16); x[3] = __uint_as_float(u.y & 0xffff0000u);
                } else {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        if (c + i < j.cols) x[i] = __uint_as_float((uint32_t)__ldg(src + i) << 16);
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) h[i] = __float_as_uint(x[i]);   // bf16 is exact in tf32
            } else {
                const float *src = static_cast<const float *>(j.X) + at;
                if (vec && c + 3 < j.cols) {
                    const float4 f = __ldg(reinterpret_cast<const float4 *>(src));
                    x[0] = f.x; x[1] = f.y; x[2] = f.z; x[3] = f.w;
                } else {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        if (c + i < j.cols) x[i] = __ldg(src + i);
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) ptx::split_tf32(x[i], h[i], l[i]);
            }
            bad |= tf32_hi_not_finite(h[0]) || tf32_hi_not_finite(h[1]) || tf32_hi_not_finite(h[2]) || tf32_hi_not_finite(h[3]);
        }
        if (!j.check_only) {
            reinterpret_cast<uint4 *>(j.hi)[g] = make_uint4(h[0], h[1], h[2], h[3]);
            if (j.lo) reinterpret_cast<uint4 *>(j.lo)[g] = make_uint4(l[0], l[1], l[2], l[3]);
        }
    }
    return bad;
}

__global__ void split_dense_kernel(SplitJobs jobs, int *__restrict__ status, TableCheck chk)
{
    ptx::launch_dependents();   // the tile kernel may take its SMs; it waits for this grid before it reads anything
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {
        if (status) *status = 0;
        if (chk.have && !signature_matches(chk.want, chk.have)) atomicExch(&chk.flags[kFlagUnsorted], 1);
    }
    bool bad = split_job(jobs.j[blockIdx.y]);
    if (jobs.has_check && blockIdx.y == 0) bad |= split_job(jobs.check);
    if (bad) atomicExch(&chk.flags[kFlagNotFinite], 1);
    if (chk.after_prepass) ptx::wait_for_primary_grid();
}

}  // namespace b2sp
