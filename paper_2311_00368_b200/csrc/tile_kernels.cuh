// Dense-tile tensor-core kernels (tcgen05 / TMEM / TMA) for SPMM over CSR with 10-30% density.
//
// Idea: at these densities a 128 x 32 window of S is a dense tile with 70-90% zeros, and the
// 5th-generation tensor cores multiply it by a dense D tile an order of magnitude faster than the
// FP32 pipes can walk its nonzeros.  fp32 accuracy is kept by splitting every operand into two
// tf32 numbers (x = hi + lo) and issuing three MMAs per product: hi*hi + lo*hi + hi*lo.
//
// Pieces:
//   tile_masks_kernel     per row and 32-column window: first CSR position + occupancy bit mask
//                         (needs strictly increasing columns in a row; sets a flag otherwise)
//   split_dense_kernel    dense fp32 operand -> zero-padded (hi, lo) tf32 copies
//   spmm_tile_kernel      one CTA per (TR-row tile of S, 128-column tile of D/O, K split): a TMA warp
//                         streams D tiles, builder warps scatter S windows into swizzled shared
//                         memory, one thread issues tcgen05.mma into a TMEM accumulator, four warps
//                         then read the accumulator back and store it
//   reduce_partials_kernel sums the K splits in fixed order
//
// Every mbarrier wait is bounded; a wait that gives up records B2SP_ERR_TIMEOUT's flag in the
// workspace status word and the CTA leaves through the normal teardown (TMEM freed).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx_sm100.cuh"

// Optional in-kernel timing of the pipeline roles (build with -DB2SP_TILE_PROFILE): per-CTA cycle
// totals are added into args.prof[0..15].
#ifdef B2SP_TILE_PROFILE
#define B2SP_PROF_DECL long long prof_t0 = 0, prof_acc[4] = {0, 0, 0, 0};
#define B2SP_PROF_START prof_t0 = clock64();
#define B2SP_PROF_STOP(i) { long long t_ = clock64(); prof_acc[i] += t_ - prof_t0; prof_t0 = t_; }
#define B2SP_PROF_FLUSH(base) { if (lane == 0 && a.prof) { for (int i_ = 0; i_ < 4; ++i_) atomicAdd(a.prof + (base) + i_, (unsigned long long)prof_acc[i_]); } }
#else
#define B2SP_PROF_DECL
#define B2SP_PROF_START
#define B2SP_PROF_STOP(i) {}
#define B2SP_PROF_FLUSH(base) {}
#endif

namespace b2sp {

constexpr int kTileKC = 32;       // columns of S per pipeline stage (one 128-byte swizzle row of tf32)
constexpr int kFlagUnsorted = 0;  // flags[0] != 0: some row's columns are not strictly increasing

// ---- table signature ------------------------------------------------------------------------------------
struct PatternSignature {
    int magic, M, K, Wk;
    long long nnz;
    const int *row_ptr, *col_idx;
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

__global__ void __launch_bounds__(kMasksWarps * 32)
tile_masks_kernel(int M, int K, int Wk, long long nnz, const int *__restrict__ row_ptr,
                  const int *__restrict__ col_idx, int2 *__restrict__ T, int *__restrict__ flags,
                  PatternSignature sig, PatternSignature *__restrict__ sig_out)
{
    extern __shared__ __align__(16) unsigned mask[];     // Wk words
    if (blockIdx.x == 0 && threadIdx.x == 0) *sig_out = sig;   // what the table is built from
    __shared__ int warp_total[kMasksWarps];
    constexpr unsigned kFull = 0xffffffffu;
    constexpr int NT = kMasksWarps * 32;
    const bool vec = (reinterpret_cast<uintptr_t>(col_idx) & 15) == 0;
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    bool bad = false;
    for (int row = blockIdx.x; row < M; row += gridDim.x) {
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
            if (w < Wk) T[(size_t)row * Wk + w] = make_int2(run + before + incl - cnt, (int)m);
            run += all;
            __syncthreads();   // warp_total and mask are reused
        }
    }
    if (bad) atomicExch(&flags[kFlagUnsorted], 1);
}

// Raises flags[kFlagUnsorted] when the workspace does not hold a table built from these arrays.
__global__ void check_signature_kernel(PatternSignature want, const PatternSignature *have, int *flags)
{
    const PatternSignature h = *have;
    if (h.magic != want.magic || h.M != want.M || h.K != want.K || h.Wk != want.Wk || h.nnz != want.nnz ||
        h.row_ptr != want.row_ptr || h.col_idx != want.col_idx)
        atomicExch(&flags[kFlagUnsorted], 1);
}

// ---- dense operand split ----------------------------------------------------------------------------
// X [rows x cols] (ld) -> hi, lo in a column-blocked layout: element (r, c) lives at
// ((c/32)*rows_p + r)*32 + c%32, i.e. [cols_p/32][rows_p][32] floats, zero in the padding
// (rows_p >= rows, cols_p >= cols, cols_p % 32 == 0).  One 32-float group of a row is one
// 128-byte swizzle row for TMA, and the whole thing is a plain packed 3-D tensor.
__global__ void split_dense_kernel(const float *__restrict__ X, long long ld, int rows, int cols,
                                   float *__restrict__ hi, float *__restrict__ lo, int rows_p, int cols_p)
{
    const long long groups = (long long)rows_p * (cols_p >> 2);  // float4 groups
    for (long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x; g < groups;
         g += (long long)gridDim.x * blockDim.x) {
        const int q = (int)(g & 7);                 // float4 inside the 32-float group
        const long long rg = g >> 3;                // (column group, row) pair
        const int r = (int)(rg % rows_p);
        const int c = (int)(rg / rows_p) * 32 + q * 4;
        uint32_t h[4] = {0, 0, 0, 0}, l[4] = {0, 0, 0, 0};
        if (r < rows) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (c + i < cols) ptx::split_tf32(__ldg(X + (long long)r * ld + c + i), h[i], l[i]);
        }
        reinterpret_cast<uint4 *>(hi)[g] = make_uint4(h[0], h[1], h[2], h[3]);
        reinterpret_cast<uint4 *>(lo)[g] = make_uint4(l[0], l[1], l[2], l[3]);
    }
}

// ---- K-split reduction ------------------------------------------------------------------------------
__global__ void reduce_partials_kernel(const float *__restrict__ part, int KS, long long slab, int ldp,
                                       int M, int N, float *__restrict__ O, long long ldo,
                                       const int *__restrict__ flags)
{
    if (flags[kFlagUnsorted] != 0) return;
    const long long total = (long long)M * N;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
         e += (long long)gridDim.x * blockDim.x) {
        int i = (int)(e / N), n = (int)(e % N);
        const float *p = part + (long long)i * ldp + n;
        float acc = p[0];
        for (int s = 1; s < KS; ++s) acc += p[(long long)s * slab];
        O[(long long)i * ldo + n] = acc;
    }
}

// ---- SPMM tile kernel ---------------------------------------------------------------------------------
// Computes O^T tiles: UMMA M = 128 columns of D/O, UMMA N = TR rows of S, K = 32 columns of S per
// stage.  A operand = D tile (MN-major tf32, streamed by TMA from the blocked hi/lo copies),
// B operand = S window tile (K-major, built here from CSR).  The streamed operand is the narrow one,
// so the L2 -> SM traffic per flop is half of what a 128-row S tile would need.
//
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer + TMEM owner, warps 2..31 = builders.  Stages
// are independent thanks to the window table, so the builders work on (stage, 16-row chunk) items
// round-robin and prefetch the records of their next item.  Builder warps 2..5 also run the epilogue.
constexpr int kTileN = 128;  // columns of D / O per CTA (UMMA M)

template <int TR>
struct SpmmTileCfg {
    static constexpr int S_BYTES = TR * kTileKC * 4;          // one S window tile (hi or lo)
    static constexpr int D_BYTES = kTileKC * kTileN * 4;      // one D tile (hi or lo): 16 KB
    static constexpr int STAGE_BYTES = 2 * S_BYTES + 2 * D_BYTES;
    static constexpr int STAGES = TR == 256 ? 2 : 3;
    static constexpr int CHUNK_ROWS = 16;                     // rows a builder warp expands per work item
    static constexpr int CHUNKS = TR / CHUNK_ROWS;            // work items per stage
    static constexpr int THREADS = 1024;                      // warp 0 TMA, warp 1 MMA, 30 builder warps
    static constexpr int BUILDERS = THREADS / 32 - 2;
    static constexpr int TMEM_COLS = TR;                      // power of two >= 32
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/ +
                                      BUILDERS * CHUNK_ROWS * 8 /*per-warp record tables*/;
};

struct SpmmTileArgs {
    int M, N, Wk, KS, Nt;
    int nnz;
    const int *col_idx;
    const float *values;
    const int2 *win;      // [M][Wk]: (first position, occupancy mask) per row and window
    float *out;           // O (KS == 1) or the partial slabs
    long long ld_out;     // leading dimension of `out`
    long long slab;       // elements between K-split slabs (0 when KS == 1)
    const int *flags;     // flags[kFlagUnsorted]
    int *status;          // device status word (set to 1 on a wait that gave up)
    unsigned long long *prof;  // optional role timers (only read when built with B2SP_TILE_PROFILE)
};

template <int TR>
__global__ void __launch_bounds__(SpmmTileCfg<TR>::THREADS, 1)
spmm_tile_kernel(const __grid_constant__ CUtensorMap tm_dhi, const __grid_constant__ CUtensorMap tm_dlo,
                 const SpmmTileArgs a)
{
    using Cfg = SpmmTileCfg<TR>;
    constexpr int STAGES = Cfg::STAGES;
    if (a.flags[kFlagUnsorted] != 0) return;  // whole grid leaves; the row kernels take over

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    const uint32_t bar_base = smem_base + STAGES * Cfg::STAGE_BYTES;
    auto full_d = [&](int s) { return bar_base + 8u * s; };
    auto full_s = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto empty = [&](int s) { return bar_base + 8u * (2 * STAGES + s); };
    const uint32_t acc_full = bar_base + 8u * (3 * STAGES);
    volatile uint32_t *tmem_slot =
        reinterpret_cast<volatile uint32_t *>(smem_gen + STAGES * Cfg::STAGE_BYTES + 8 * (3 * STAGES + 1));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // work item
    const int ks = blockIdx.x % a.KS;
    const int tile = blockIdx.x / a.KS;
    const int nt = tile % a.Nt, mt = tile / a.Nt;
    const int w0 = (int)((long long)a.Wk * ks / a.KS), w1 = (int)((long long)a.Wk * (ks + 1) / a.KS);
    const int nchunks = w1 - w0;
    const int m0 = mt * TR, n0 = nt * kTileN;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(full_d(s), 1);
            ptx::mbar_init(full_s(s), Cfg::CHUNKS);
            ptx::mbar_init(empty(s), 1);
        }
        ptx::mbar_init(acc_full, 1);
        ptx::fence_mbar_init();
    }
    if (warp == 1) {
        __syncwarp();
        ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t *>(tmem_slot)), Cfg::TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_acc = *tmem_slot;
    bool failed = false;

    if (warp == 0) {
        // ---------------- TMA producer: D_hi / D_lo tiles ----------------
        if (lane == 0) {
            ptx::tma_prefetch_desc(&tm_dhi);
            ptx::tma_prefetch_desc(&tm_dlo);
            int issued = 0;
            B2SP_PROF_DECL
            B2SP_PROF_START
            for (int it = 0; it < nchunks; ++it) {
                const int s = it % STAGES;
                if (it >= STAGES && !ptx::mbar_wait(empty(s), ((it / STAGES) - 1) & 1)) { failed = true; break; }
                B2SP_PROF_STOP(0)
                const uint32_t dst = smem_base + s * Cfg::STAGE_BYTES + 2 * Cfg::S_BYTES;
                ptx::mbar_arrive_expect_tx(full_d(s), 2 * Cfg::D_BYTES);
                ptx::tma_load_3d(dst, &tm_dhi, full_d(s), 0, (w0 + it) * kTileKC, nt * (kTileN / 32));
                ptx::tma_load_3d(dst + Cfg::D_BYTES, &tm_dlo, full_d(s), 0, (w0 + it) * kTileKC, nt * (kTileN / 32));
                issued = it + 1;
                B2SP_PROF_STOP(1)
            }
            B2SP_PROF_FLUSH(0)
            if (failed) {  // let the copies already in flight land before the CTA goes away
                for (int it = issued > STAGES ? issued - STAGES : 0; it < issued; ++it)
                    ptx::mbar_wait(full_d(it % STAGES), (it / STAGES) & 1);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            // A = D tile: MN-major; B = S tile: K-major
            constexpr uint32_t idesc = ptx::idesc_tf32(kTileN, TR, /*a_mn_major=*/true, /*b_mn_major=*/false);
            B2SP_PROF_DECL
            B2SP_PROF_START
            for (int it = 0; it < nchunks; ++it) {
                const int s = it % STAGES;
                const uint32_t par = (it / STAGES) & 1;
#ifdef B2SP_PROF_DFIRST
                if (!ptx::mbar_wait(full_d(s), par)) { failed = true; break; }
                B2SP_PROF_STOP(1)
                if (!ptx::mbar_wait(full_s(s), par)) { failed = true; break; }
                B2SP_PROF_STOP(0)
#else
                if (!ptx::mbar_wait(full_s(s), par)) { failed = true; break; }
                B2SP_PROF_STOP(0)
                if (!ptx::mbar_wait(full_d(s), par)) { failed = true; break; }
                B2SP_PROF_STOP(1)
#endif
                ptx::tc_fence_after_sync();
                const uint32_t s_hi = smem_base + s * Cfg::STAGE_BYTES, s_lo = s_hi + Cfg::S_BYTES;
                const uint32_t d_hi = s_lo + Cfg::S_BYTES, d_lo = d_hi + Cfg::D_BYTES;
#pragma unroll
                for (int k8 = 0; k8 < kTileKC / 8; ++k8) {
                    // S: K-major, 128-byte swizzle rows, 8-row groups 1024 B apart; +32 B per K step of 8
                    const uint64_t b_hi = ptx::smem_desc(s_hi + k8 * 32, 16, 1024, ptx::kLayoutSw128);
                    const uint64_t b_lo = ptx::smem_desc(s_lo + k8 * 32, 16, 1024, ptx::kLayoutSw128);
                    // D: MN-major tf32 (128-byte swizzle in 32-byte units): 32-float column groups
                    // kTileKC*128 B apart, 4-row K groups 512 B apart; +1024 B per K step of 8 rows
                    const uint64_t a_hi = ptx::smem_desc(d_hi + k8 * 1024, kTileKC * 128, 512, ptx::kLayoutSw128Base32);
                    const uint64_t a_lo = ptx::smem_desc(d_lo + k8 * 1024, kTileKC * 128, 512, ptx::kLayoutSw128Base32);
                    ptx::mma_tf32_ss(tmem_acc, a_hi, b_hi, idesc, (it | k8) != 0);
                    ptx::mma_tf32_ss(tmem_acc, a_hi, b_lo, idesc, 1);
                    ptx::mma_tf32_ss(tmem_acc, a_lo, b_hi, idesc, 1);
                }
                ptx::mma_commit(empty(s));
                B2SP_PROF_STOP(2)
            }
            B2SP_PROF_FLUSH(4)
            if (!failed) ptx::mma_commit(acc_full);
        }
    } else {
        // ---------------- builders: expand S windows into swizzled K-major tiles ----------------
        // Work item = (stage, chunk of 16 rows); the builder warps take items round-robin, so the 16
        // chunks of a stage are expanded by 16 different warps at once and later stages are already
        // in progress.  Inside an item a lane owns one column of the 32-column window: lanes 0..15
        // first fetch (position, mask) of the chunk's rows (one item ahead) and park them in a small
        // shared table; then, row by row, lane c reads the row's entry through the warp-uniform
        // mask: present iff bit c is set, stored at position + popc(mask below c).  Every lane writes
        // its element (value or 0) of every row, so the tile needs no separate clearing and col_idx
        // is never read here.  hi = value rounded to tf32, lo = value - hi (exact; the tensor core
        // keeps its leading tf32 bits).
        constexpr int CR = Cfg::CHUNK_ROWS, CH = Cfg::CHUNKS, NB = Cfg::BUILDERS;
        const int b = warp - 2;
        const uint32_t tab = smem_base + STAGES * Cfg::STAGE_BYTES + 256 + b * (CR * 8);   // shared address
        const unsigned lane_bit = 1u << lane, lt_mask = lane_bit - 1u;
        const int nitems = nchunks * CH;
        auto record = [&](int id) {                    // lanes 0..15: window record of one row of item `id`
            int2 rec = make_int2(0, 0);
            const int row = m0 + (id % CH) * CR + lane;
            if (id < nitems && lane < CR && row < a.M) rec = __ldg(a.win + (size_t)row * a.Wk + w0 + id / CH);
            return rec;
        };
        int2 nxt = record(b);
        B2SP_PROF_DECL
        B2SP_PROF_START
        for (int id = b; id < nitems; id += NB) {
            const int it = id / CH, chunk = id % CH, slot = it % STAGES, use = it / STAGES;
            __syncwarp();   // everyone is done with the previous item's table
            if (lane < CR) ptx::sts64(tab + lane * 8, (uint32_t)nxt.x, (uint32_t)nxt.y);
            nxt = record(id + NB);
            __syncwarp();
            float x[CR];
            ptx::for_each_row<CR>([&](auto rc) {
                constexpr int r = decltype(rc)::value;
                uint32_t pos, mask;
                ptx::lds64_off<r * 8>(tab, pos, mask);
                x[r] = 0.f;
#ifdef B2SP_ABL_NOLOAD
                if (mask & lane_bit) x[r] = __uint_as_float(pos + __popc(mask & lt_mask));
#else
                if (mask & lane_bit) x[r] = __ldg(a.values + (pos + __popc(mask & lt_mask)));
#endif
            });
            B2SP_PROF_STOP(0)
            {   // the slot must have been drained by the MMAs of its previous use
                bool ok = use == 0 || ptx::mbar_wait(empty(slot), (use - 1) & 1);
                if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
            }
            B2SP_PROF_STOP(1)
            // shared address of this lane's column in row r of the chunk: wb[r & 7] + r * 128
            const uint32_t w_hi = smem_base + slot * Cfg::STAGE_BYTES + chunk * (CR * 128);
            uint32_t wb[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) wb[i] = w_hi + (uint32_t)((lane << 2) ^ (i << 4));
            ptx::for_each_row<CR>([&](auto rc) {
                constexpr int r = decltype(rc)::value;
                const uint32_t hi = (__float_as_uint(x[r]) + 0x1000u) & 0xffffe000u;
                const float lo = x[r] - __uint_as_float(hi);
#ifdef B2SP_ABL_NOSTORE
                if (hi == 0x12345678u)
#endif
                {
                    ptx::sts32_off<r * 128>(wb[r & 7], hi);
                    ptx::sts32_off<r * 128 + Cfg::S_BYTES>(wb[r & 7], __float_as_uint(lo));
                }
            });
            B2SP_PROF_STOP(2)
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(full_s(slot));
            B2SP_PROF_STOP(3)
        }
        if (b < 2) { B2SP_PROF_FLUSH(8) }
        // ---------------- epilogue (first four builder warps): accumulator -> global ----------------
        if (warp < 6) {
            {
                bool ok = !failed && ptx::mbar_wait(acc_full, 0);
                failed = !__all_sync(0xffffffffu, ok);
            }
            if (!failed) {
                ptx::tc_fence_after_sync();
                const int q = warp & 3;                 // TMEM lane quarter this warp may access
                const int n = n0 + q * 32 + lane;       // O column held by this lane
                float *obase = a.out + (long long)ks * a.slab + n;
#pragma unroll 1
                for (int c = 0; c < TR / 32; ++c) {
                    uint32_t r[32];
                    ptx::tmem_ld_32x32(tmem_acc + ((uint32_t)(q * 32) << 16) + c * 32, r);
                    ptx::tmem_ld_wait();
                    if (n < a.N) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            const int row = m0 + c * 32 + i;
                            if (row < a.M) obase[(long long)row * a.ld_out] = __uint_as_float(r[i]);
                        }
                    }
                }
            }
        }
    }
    if (failed) atomicExch(a.status, 1);
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        ptx::tmem_dealloc(tmem_acc, Cfg::TMEM_COLS);
    }
}

}  // namespace b2sp
