// Dense-tile FusedMM, SDDMM and SPMM (tcgen05 / TMEM / TMA, 3xTF32) over the window table of S:
// one kernel, three modes.
//
// One CTA owns 128 rows of S (= rows of A and O), a range of 128-column blocks of S (4 windows of 32
// columns each) and, for FusedMM / SPMM, one 128-column tile of O -- or, on the balanced partition (see
// kFusedMaxSegs), a run of blocks that may go on from one row tile into the next ones.
//   * A_tile (128 x Kd) is split into tf32 hi/lo once: A_hi lives in tensor memory for the CTA's
//     life; A_lo lives in tensor memory too (SDDMM) or in shared memory (FusedMM, where TMEM is
//     needed for O and P').
//   * Per block: GEMM1  P = A_tile * B_block^T  (128 x 128).  The B rows of the block arrive by TMA
//     in chunks of 32 k (hi + lo, 32 KB); N = 128 MMAs run the tensor pipe at full rate (a 128xNx8
//     tf32 MMA costs max(N/2, 45.6) cycles, so 32-column GEMMs would waste two thirds of it).
//   * Four processor warps (thread = row) read P window by window (32 columns) and multiply it by the
//     window's stored values (0 where nothing is stored), which helper warps fetch with lane =
//     column (coalesced), densify and transpose through shared-memory slots.  The sampled C of the
//     paper (Alg. 3) exists only in these registers.  Then
//       - FusedMM: split the result into hi/lo and write it back to TMEM as P' (two buffers); GEMM2
//         O += P'_window * D_window (A = P' from TMEM, B = D rows by TMA, MN-major) accumulates O in TMEM;
//       - SDDMM (Alg. 1): the processors hand their rows of P to the helpers through the slots; the
//         helpers multiply by the stored values and write each row's entries as one contiguous run.
//   * SPMM (Alg. 2) is the FusedMM pipeline with P' = the stored values themselves: no A, no B, no GEMM1.
//
// TMEM columns (512 allocated)
//   FusedMM: O [0,128)  P [128,256)  P'0 hi/lo [256,288)/[288,320)  P'1 hi/lo [320,352)/[352,384)  A_hi [384,384+Kdp)
//   SPMM:    O0 [0,128)  O1 [128,256)  P' as for FusedMM
//   SDDMM:   P0 [0,128) P1 [128,256) A_hi [256,256+Kdp)  A_lo [384,384+Kdp)
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx_sm100.cuh"
#include "slab_sum.cuh"
#include "tile_kernels.cuh"


namespace b2sp {

constexpr int kFusedRows = 128;     // rows per CTA (UMMA M)
constexpr int kFusedW = 32;         // S columns per window
constexpr int kFusedBlk = 128;      // S columns per block (UMMA N of GEMM1)
// FusedMM and SPMM: 20 warps = 5 per scheduler (a sixth would cut the register budget from 96 to 80 per
// thread; measured slower).  Warp 1: MMA issue + TMEM owner; warp 9: TMA producer; warps 2-5: processors;
// warps 16-19: second processor set (FusedMM) or flusher warps (SPMM); helpers among warps 0, 6-8, 10-15
// (FusedMM: eight, none on the MMA warp's scheduler, warps 13 and 15 idle; SPMM: ten, warp 13 included).
// SDDMM: 28 warps of 72 registers, see FusedCfg.
constexpr int kFusedThreads = 640;
constexpr int kFusedTmaWarp = 9;
constexpr int kFusedMaxHelpers = 20;
constexpr int kFusedNT = 128;       // most O columns per CTA (UMMA N of GEMM2); see FusedTileArgs::NT
// The tensor core adds every MMA into its fp32 accumulator with truncation: a bias of about -2e-8 of
// the running sum per MMA, which nothing cancels on same-sign data (measured: -3.0e-5 after the 1536
// MMAs of 32 blocks, three times the 1e-5 gate).  So O is accumulated in tensor memory over at most
// kFusedFlushBlocks blocks (192 MMAs, bias <= 4e-6), then added into the output in global memory with
// round-to-nearest fp32 reductions and restarted from zero.
constexpr int kFusedFlushBlocks = 4;
constexpr int kFusedChunk = 32768;  // bytes of one pipeline chunk (hi + lo)
// The balanced partition (FusedTileArgs::bal_ctas): the CTAs form groups of Nt (one CTA per column tile of O), and
// the granules of all row tiles -- the 4-block flush granules of FusedMM / SPMM, single blocks for SDDMM -- in the order
// (problem, row tile, granule) are dealt evenly to the groups: group c of n gets granules [c * G / n, (c + 1) * G / n)
// of G.  So a CTA may finish one output tile and go on with the next row tile's: at most kFusedMaxSegs segments, each
// (FusedMM / SPMM) with a slab of its own (the tile's first, second, ... segment writes slab 0, 1, ...); between
// segments FusedMM and SDDMM reload their A tile.  The CTAs of a group work on the same blocks of S at the same time,
// so S is fetched from memory once per group.
// (struct Balance, in slab_sum.cuh, holds the arithmetic.)
constexpr int kFusedMaxSegs = 4;

struct FusedTileArgs {
    int M, K, Kd, Kdp, N, Wk, KS, Nt;
    // A batch of `batch` independent problems of the same sizes in one launch: CTA blockIdx.x works on problem
    // blockIdx.x / ctas_per_problem.  Window tables, tf32 operand copies (rows b*Kp ...) and slabs of the problems
    // are stacked; the caller's arrays are `stride_*` elements apart.
    int batch, ctas_per_problem, Kp;
    long long stride_sv, stride_A, stride_O;
    int NT;                   // O columns per CTA (UMMA N of GEMM2): 128, or 64 when N <= 64
    int tiles_pp;             // output tiles per problem (row tiles x column tiles)
    int bal_ctas;             // > 0: the balanced partition over this many CTAs (KS = slabs per tile then); 0: every
                              // CTA has one tile and one of its KS equal K splits
    const int2 *win;          // [M][Wk] window records (position, mask)
    const float *s_values;    // NULL = all ones
    const void *A;            // M x Kd, fp32 (bfloat16 in the EXACT kernels)
    long long lda;
    float *out;               // FusedMM / SPMM: O (one K split) or the K splits' slabs; SDDMM: out_values
    long long ld_out, slab;
    int out_tma;              // the flush may use TMA on `out` (tm_out covers it; 16-byte aligned rows)
    int slab_rows;            // rows of one slab (TMA y coordinate of slab ks = ks * slab_rows)
    float *O;                 // the caller's output (several slabs per tile: the grid behind this one adds them into it, see slab_sum.cuh)
    long long ldo;
    int *flags;                // flags[kFlagUnsorted] or flags[kFlagNotFinite] != 0: the row kernels take over
    int *status;
    int debug_drop_chunk;      // test hook: the TMA producer leaves out this chunk of every CTA (-1: none), so that the
                               // waits for it run out and the CTA reports B2SP_ERR_TIMEOUT through the status word
};

// MODE: which op the kernel runs.  SPMM reuses the FusedMM pipeline with P' = the stored values
// themselves (no A, no GEMM1).
constexpr int kModeSddmm = 0, kModeFused = 1, kModeSpmm = 2;

// Which helper a warp is (-1: none).  20-warp kernels (FusedMM, SPMM): warps 0, 6, 7, 8, 10, 11, 12, 14, 15
// -> 0 .. 8 (none on the MMA warp's scheduler, warp % 4 == 1), then warp 13 -> 9; warps 16-19 have other roles.
// 28-warp kernel (SDDMM): every warp but 1-5 (MMA, processors), 9 (TMA), 21 and 25.
template <bool NARROW>
__device__ __forceinline__ int helper_index(int warp)
{
    if (NARROW) return warp == 13 ? 9 : (warp & 3) == 1 || (warp >= 2 && warp < 6) || warp >= 16 ? -1 : warp == 0 ? 0 : 1 + (warp - 6) - ((warp - 5) >> 2);
    if ((warp >= 1 && warp < 6) || warp == 9 || warp == 21 || warp == 25) return -1;
    return warp == 0 ? 0 : 1 + (warp - 6) - (warp > 9 ? 1 : 0) - (warp > 21 ? 1 : 0) - (warp > 25 ? 1 : 0);
}

// EXACT: the dense operands A, B, D are exact in tf32 (bfloat16 inputs): their lo halves are zero, so the lo
// copies are neither loaded nor multiplied -- GEMM1 is one MMA per product instead of three, GEMM2 two (P' still
// has a hi and a lo part).
template <int KDP, int MODE, bool EXACT = false>
struct FusedCfg {
    static constexpr bool FUSED = MODE != kModeSddmm;          // has GEMM2 / O
    static constexpr bool SPMM = MODE == kModeSpmm;
    static constexpr int NCH_B = SPMM ? 0 : KDP / 32;          // B chunks per block
    static constexpr int NCH_D = FUSED ? kFusedBlk / kFusedW : 0;  // D chunks per block
    static constexpr int ALO_BYTES = (FUSED && !SPMM && !EXACT) ? kFusedRows * KDP * 4 : 0;
    // SDDMM runs 28 warps of 72 registers (its processors only copy P, and its helpers work on items of
    // 16 rows, so nobody needs more) with twenty helpers.  FusedMM and SPMM: 20 warps of 96.
    // SPMM has four flusher warps (16-19) of its own: it has two O accumulators so that the tensor core can go on
    // while a partial sum leaves tensor memory, which only helps if the processors, who make its next operands,
    // are not the ones doing the flush (measured with role timers: a third of the processors' time).
    static constexpr bool DEDICATED_FLUSH = SPMM;
    static constexpr int THREADS = !FUSED ? 896 : kFusedThreads;
    static constexpr int FLUSH_WARP0 = 16;   // the flusher warps: 16-19 (SPMM: dedicated; FusedMM: the second processor set)
    static constexpr int RING = FUSED ? 3 : 4;   // TMA chunks in flight (32 KB each)
    // FusedMM is bound by the tensor pipe and its helpers are mostly idle: eight of them, with eight
    // 4 KB slots (two windows deep).  SPMM, whose helpers are the bound: the ten warps left beside the flusher
    // warps, with twenty slots.  SDDMM: twenty with forty 2 KB slots (measured: 12 helpers 134 us, 14 helpers
    // 129 us, 20 helpers on 28 warps 125 us; for SPMM the 28-warp layout was slower, 136-140 us against 131 us).
    static constexpr int HELPERS = SPMM ? 10 : FUSED ? 8 : 20;
    // FusedMM runs two sets of processor warps (warps 2-5 and 16-19) that take alternate windows: a window is a
    // chain of long-latency steps for its processor (slot, tensor-memory load, arithmetic, tensor-memory store,
    // hand-over), about 2 k cycles, and with a single set that chain, not the tensor core, paced the kernel
    // wherever a window holds less than 2 k cycles of MMAs.  The second set (odd windows) also does the flushes.
    static constexpr int PSETS = (FUSED && !SPMM) ? 2 : 1;
    static constexpr int ITEM_ROWS = FUSED ? 32 : 16;           // rows of a helper's work item
    static constexpr int IPW = kFusedRows / ITEM_ROWS;         // items per window
    static constexpr int SLOT_BYTES = ITEM_ROWS * 128;
    static constexpr int SLOTS = SPMM ? 20 : FUSED ? HELPERS : 2 * HELPERS;
    // A slot's mbarriers are waited on by parity, which is only sound when the waiter is at most one
    // phase away: every slot is always filled by the same helper and drained by the same processor warp.
    static_assert(SLOTS % HELPERS == 0 && SLOTS % IPW == 0, "slot ownership must be fixed");
    static constexpr int FLUSH_BYTES = FUSED ? 4 * 4096 : 0;   // per flushing warp: two buffers of 32 rows x 16 columns
    static constexpr int AUX_BYTES = 1024 /*barriers*/ + kFusedMaxHelpers * 256 /*record tables*/ + SLOTS * SLOT_BYTES + FLUSH_BYTES;
    static constexpr int SMEM_BYTES = RING * kFusedChunk + ALO_BYTES + 1024 + AUX_BYTES;
    // tensor-memory columns
    // SPMM has tensor memory to spare: two O accumulators, so that the tensor core works on the next
    // chunk of blocks while the previous partial sum is flushed.
    static constexpr int NOB = SPMM ? 2 : 1;
    // the balanced partition deals granules of this many blocks: the flush granules of FusedMM / SPMM, single blocks for SDDMM
    static constexpr int GRAN = FUSED ? kFusedFlushBlocks : 1;
    static constexpr uint32_t COL_O = 0, COL_P = FUSED ? 128 : 0, COL_PP = 256;
    static constexpr uint32_t COL_AHI = FUSED ? 384 : 256, COL_ALO = 384;
};

// One thread's row (`row` of the tile, tensor-memory lane address lane_addr) of the A tile that begins at row tm0 of
// problem tprob: the 16-column groups first, first + step, ... are split into tf32 hi (tensor memory) and lo (tensor
// memory for SDDMM, shared memory at alo_smem for FusedMM; none for operands exact in tf32).
template <int KDP, int MODE, bool EXACT>
__device__ __forceinline__ void load_a_tile_impl(const void *A, long long lda, long long stride_A, int M, int Kd, uint32_t tmem,
                                                 uint32_t lane_addr, uint32_t alo_smem, int row, int tm0, int tprob, int first, int step)
{
    using Cfg = FusedCfg<KDP, MODE, EXACT>;
    constexpr bool FUSED = Cfg::FUSED;
    struct { const void *A; long long lda, stride_A; int M, Kd; } a = {A, lda, stride_A, M, Kd};

        const int grow = tm0 + row;
        const long long aoff = tprob * a.stride_A + (long long)(grow < a.M ? grow : 0) * a.lda;
        const float *arow = static_cast<const float *>(a.A) + aoff;
        const unsigned short *arow16 = static_cast<const unsigned short *>(a.A) + aoff;
        const bool vec = (a.lda & 3) == 0 && (a.stride_A & 3) == 0 && (reinterpret_cast<uintptr_t>(a.A) & 15) == 0 &&
                         (!EXACT || (a.lda & 7) == 0);   // (16-byte loads of eight bf16)
#pragma unroll 1
        for (int c = first * 16; c < KDP; c += step * 16) {
            uint32_t hi[16], lo[16];
            float v[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = 0.f;
            if (grow < a.M) {
                if (EXACT) {
                    if (vec && c + 16 <= a.Kd) {
#pragma unroll
                        for (int i = 0; i < 16; i += 8) {
                            const uint4 u = __ldg(reinterpret_cast<const uint4 *>(arow16 + c + i));
                            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                v[i + 2 * j] = __uint_as_float(w[j] << 16);
                                v[i + 2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
                            }
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            if (c + i < a.Kd) v[i] = __uint_as_float((uint32_t)__ldg(arow16 + c + i) << 16);
                    }
                } else if (vec && c + 16 <= a.Kd) {
#pragma unroll
                    for (int i = 0; i < 16; i += 4) {
                        const float4 f = __ldg(reinterpret_cast<const float4 *>(arow + c + i));
                        v[i] = f.x; v[i + 1] = f.y; v[i + 2] = f.z; v[i + 3] = f.w;
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (c + i < a.Kd) v[i] = __ldg(arow + c + i);
                }
            }
            if constexpr (EXACT) {   // the value is its own hi part
#pragma unroll
                for (int i = 0; i < 16; ++i) hi[i] = __float_as_uint(v[i]);
                ptx::tmem_st_32x16(tmem + lane_addr + Cfg::COL_AHI + c, hi);
            } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) ptx::split_tf32_fast(v[i], hi[i], lo[i]);
            ptx::tmem_st_32x16(tmem + lane_addr + Cfg::COL_AHI + c, hi);
            if (FUSED) {
                // K-major, 128-byte swizzle: 16 KB sub-tile per 32 k, row = 128 B, 16-byte chunk j at j ^ (row & 7)
                const uint32_t base = alo_smem + (c >> 5) * (kFusedRows * 128) + row * 128;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t chunk = (uint32_t)(((c & 31) >> 2) + j);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(base + ((chunk ^ (row & 7)) << 4)),
                                 "r"(lo[4 * j]), "r"(lo[4 * j + 1]), "r"(lo[4 * j + 2]), "r"(lo[4 * j + 3]) : "memory");
                }
            } else {
                ptx::tmem_st_32x16(tmem + lane_addr + Cfg::COL_ALO + c, lo);
            }
            }
        }
        ptx::tmem_st_wait();
        if (FUSED) ptx::fence_proxy_async_smem();
    }

// The same as a function of its own, for the reload at the end of a segment of the balanced partition: it runs once per
// segment, and its code stays out of the processors' loop.
template <int KDP, int MODE, bool EXACT>
__device__ __noinline__ void reload_a_tile(const void *A, long long lda, long long stride_A, int M, int Kd, uint32_t tmem,
                                           uint32_t lane_addr, uint32_t alo_smem, int row, int tm0, int tprob)
{
    load_a_tile_impl<KDP, MODE, EXACT>(A, lda, stride_A, M, Kd, tmem, lane_addr, alo_smem, row, tm0, tprob, 0, 1);
}

// PART: how the work is dealt to CTAs.  kPartTiles: every CTA has one output tile and one of its KS equal K splits.
// kPartBatched: the same over several problems (FusedTileArgs::batch) -- a template parameter because without it the
// problem index is the constant 0 and the kernel is exactly the single-problem one (the SDDMM mode has no registers to
// spare).  kPartBalanced: the balanced partition (see kFusedMaxSegs); a template parameter too: with the choice made
// at run time the SPMM kernel was 5% slower on either partition.
constexpr int kPartTiles = 0, kPartBatched = 1, kPartBalanced = 2;
template <int KDP, int MODE, int PART = kPartTiles, bool EXACT = false>
__global__ void __launch_bounds__((FusedCfg<KDP, MODE, EXACT>::THREADS), 1)
fused_tile_kernel(const __grid_constant__ CUtensorMap tm_bhi, const __grid_constant__ CUtensorMap tm_blo,
                  const __grid_constant__ CUtensorMap tm_dhi, const __grid_constant__ CUtensorMap tm_dlo,
                  const __grid_constant__ CUtensorMap tm_out, const FusedTileArgs a)
{
    using Cfg = FusedCfg<KDP, MODE, EXACT>;
    constexpr bool FUSED = Cfg::FUSED, SPMM = Cfg::SPMM;
    constexpr int RING = Cfg::RING, NCH_B = Cfg::NCH_B;
    constexpr int WPB = kFusedBlk / kFusedW;   // windows per block
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    const uint32_t ring = smem_base;                               // RING chunks of 32 KB
    const uint32_t alo_smem = smem_base + RING * kFusedChunk;      // FusedMM: A_lo, K-major, 16 KB per 32 k
    const uint32_t aux = alo_smem + Cfg::ALO_BYTES;
    auto full = [&](int s) { return aux + 8u * s; };
    auto empty = [&](int s) { return aux + 8u * (RING + s); };
    auto p_full = [&](int b) { return aux + 8u * (2 * RING + b); };
    auto p_free = [&](int b) { return aux + 8u * (2 * RING + 2 + b); };
    auto pp_full = [&](int b) { return aux + 8u * (2 * RING + 4 + b); };
    auto pp_free = [&](int b) { return aux + 8u * (2 * RING + 6 + b); };
    constexpr int NSLOT = Cfg::SLOTS, NH = Cfg::HELPERS, NOB = Cfg::NOB;
    auto o_full = [&](int b) { return aux + 8u * (b == 0 ? 2 * RING + 8 : 2 * RING + 11 + 2 * NSLOT); };
    auto sl_full = [&](int s) { return aux + 8u * (2 * RING + 9 + s); };
    auto sl_empty = [&](int s) { return aux + 8u * (2 * RING + 9 + NSLOT + s); };
    auto o_free = [&](int b) { return aux + 8u * (2 * RING + 9 + 2 * NSLOT + b); };
    const uint32_t a_ready = aux + 880;   // balanced FusedMM: the A tile of the next segment is in place (four processor warps)
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem_gen + (aux - smem_base) + 8 * (2 * RING + 12 + 2 * NSLOT));
    const uint32_t helper_tabs = aux + 1024, slots = aux + 1024 + kFusedMaxHelpers * 256;
    const uint32_t flush_stage = slots + NSLOT * Cfg::SLOT_BYTES;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr bool BATCHED = PART == kPartBatched, bal = PART == kPartBalanced;
    const int prob = BATCHED ? blockIdx.x / a.ctas_per_problem : 0;            // problem of the batch
    const int cta = BATCHED ? blockIdx.x % a.ctas_per_problem : blockIdx.x;
    const int ks = cta % a.KS;
    const int tile = cta / a.KS;
    const int nt = tile % a.Nt, mt = tile / a.Nt;
    const int nblk_all = (a.Wk + WPB - 1) / WPB;
    const int m0 = mt * kFusedRows;
    const int tiles_pp = a.tiles_pp;                             // output tiles per problem
    const int krow0 = prob * a.Kp;                               // first row of this problem in the stacked operand copies
    // Balanced partition: this CTA's granules [g0, g1) of the batch's units * gpt, and its segments (one per
    // output tile it touches) in shared memory, read by the roles through seg_at().
    // segment records of eight ints (first block counted from the CTA's first, first row of the tile, column tile,
    // first block within the tile's row of blocks, slab, problem, -, -); their number at segtab - 8
    const uint32_t segtab = aux + 896;
    constexpr uint32_t kSegStart = 0, kSegM0 = 4, kSegNt = 8, kSegBt0 = 12, kSegOrd = 16, kSegProb = 20;
    constexpr int GRAN = Cfg::GRAN;
    const int gpt = nblk_all / GRAN;
    const int grp = (int)blockIdx.x / a.Nt;                        // (CTA blockIdx.x: group grp, column tile blockIdx.x % Nt)
    const int mtiles = tiles_pp / a.Nt;                            // row tiles per problem
    const Balance balance(bal ? a.batch * mtiles * gpt : 1, bal ? a.bal_ctas / a.Nt : 1);
    const int g0 = bal ? balance.start(grp) : 0, g1 = bal ? balance.start(grp + 1) : 0;
    const int b0 = bal ? 0 : nblk_all * ks / a.KS;   // (32-bit: at most 6 k blocks, 32 splits)
    const int nblk = bal ? (g1 - g0) * GRAN : nblk_all * (ks + 1) / a.KS - b0;
    if (bal && threadIdx.x == 0) {
        int n = 0;
        for (int g = g0; g < g1 && n < kFusedMaxSegs; ++n) {
            const int unit = g / gpt;                    // problem * row tiles + row tile
            const int gfirst = unit * gpt;
            const uint32_t rec = segtab + n * 32;
            ptx::sts32(rec + kSegStart, (uint32_t)((g - g0) * GRAN));
            ptx::sts32(rec + kSegM0, (uint32_t)(unit % mtiles * kFusedRows));
            ptx::sts32(rec + kSegNt, (uint32_t)((int)blockIdx.x % a.Nt));
            ptx::sts32(rec + kSegBt0, (uint32_t)((g - gfirst) * GRAN));
            ptx::sts32(rec + kSegOrd, (uint32_t)(grp - balance.group_of(gfirst)));
            ptx::sts32(rec + kSegProb, (uint32_t)(unit / mtiles));
            g = gfirst + gpt < g1 ? gfirst + gpt : g1;
        }
        ptx::sts32(segtab - 8, (uint32_t)n);
    }
    // the record (shared-memory address) of the segment that holds block blk of this CTA, and a field of a record
    auto seg_at = [&](int blk) -> uint32_t {
        const int n = (int)ptx::lds32(segtab - 8);
        uint32_t rec = segtab;
        for (int i = 1; i < n; ++i) rec += blk >= (int)ptx::lds32(segtab + i * 32) ? 32u : 0u;
        return rec;
    };
    auto seg_f = [&](uint32_t rec, uint32_t field) -> int { return (int)ptx::lds32(rec + field); };

    if (threadIdx.x == 0) {
        for (int s = 0; s < RING; ++s) { ptx::mbar_init(full(s), 1); ptx::mbar_init(empty(s), 1); }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(p_full(b), 1);
            ptx::mbar_init(p_free(b), FUSED ? 4 * Cfg::PSETS : 4);
            ptx::mbar_init(pp_full(b), 4);
            ptx::mbar_init(pp_free(b), 1);
        }
        for (int b = 0; b < NOB; ++b) { ptx::mbar_init(o_full(b), 1); ptx::mbar_init(o_free(b), 4); }
        for (int s = 0; s < NSLOT; ++s) { ptx::mbar_init(sl_full(s), 1); ptx::mbar_init(sl_empty(s), 1); }
        ptx::mbar_init(a_ready, 4);
        ptx::fence_mbar_init();
    }
    if (warp == 1) {
        __syncwarp();
        ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t *>(tmem_slot)), 512);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    bool failed = false;

    // ---- A tile -> TMEM (hi, and lo for SDDMM) / shared memory (lo for FusedMM); thread = row ----
    // A warp reaches the tensor-memory lanes of quarter warp % 4: all warps of a quarter but the MMA and the
    // TMA warp share the tile's 16-column groups.
    const int q = warp & 3;                 // TMEM lane quarter
    const int row = q * 32 + lane;          // row inside the tile
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    constexpr int NWARP = Cfg::THREADS / 32;
    const int pro_n = q == 1 ? NWARP / 4 - 2 : NWARP / 4;                            // warps of this quarter that take part
    const int pro_i = q == 1 ? (warp == 5 ? 0 : (warp >> 2) - 2) : (warp >> 2);      // ... and this warp's place among them
    if (!SPMM && warp != 1 && warp != kFusedTmaWarp)
        load_a_tile_impl<KDP, MODE, EXACT>(a.A, a.lda, a.stride_A, a.M, a.Kd, tmem, lane_addr, alo_smem, row, bal ? (int)ptx::lds32(segtab + kSegM0) : m0,
                                           bal ? (int)ptx::lds32(segtab + kSegProb) : prob, pro_i, pro_n);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();

    // Everything above (barriers, tensor memory, the A tile: none of it written by the kernel before) ran
    // while the operand-split kernel, whose programmatic dependent this grid is, was still at work.  Its tf32
    // copies and its check of a prepared table are needed from here on.  After it the flags are final (the
    // pre-pass or that kernel's signature check wrote them), so the gated row kernel launched behind this
    // grid may run beside it.
    ptx::wait_for_primary_grid();
    const bool unusable = (a.flags[kFlagUnsorted] | a.flags[kFlagNotFinite]) != 0;
    ptx::launch_dependents();
    if (unusable) {   // pattern not usable for tiles: the row kernels take over
        if (warp == 1) {
            __syncwarp();
            ptx::tmem_dealloc(tmem, 512);
        }
        return;
    }

    // ---- flush of one chunk of blocks: the partial O leaves tensor memory.  Called by the four warps (one per
    // tensor-memory lane quarter q) that do the flushes: each thread adds its row into the output (or its K
    // split's slab): the first partial sum is stored, the later ones are added with fp32 reductions (round to
    // nearest).  A given element is only ever touched by the same lane of the same warp, in program order, so
    // the sum is reproducible.  false: a bounded wait gave up.
    auto flush_chunk = [&](int chunk) -> bool {
        const int ob = chunk % NOB;
        // the tile the chunk belongs to, its slab, and whether the chunk is the first partial sum that goes there
        int m0 = mt * kFusedRows, n0 = nt * a.NT, ks = cta % a.KS, prob = BATCHED ? blockIdx.x / a.ctas_per_problem : 0;
        bool first_sum = chunk == 0;
        if (bal) {
            const uint32_t sg = seg_at(chunk * kFusedFlushBlocks);
            m0 = seg_f(sg, kSegM0); n0 = seg_f(sg, kSegNt) * a.NT; ks = seg_f(sg, kSegOrd); prob = seg_f(sg, kSegProb);
            first_sum = chunk * kFusedFlushBlocks == seg_f(sg, kSegStart);
        }
        const bool cat_halves = !EXACT && a.NT == 64;
        bool ok = ptx::mbar_wait(o_full(ob), (chunk / NOB) & 1);
        if (!__all_sync(0xffffffffu, ok)) return false;
        ptx::tc_fence_after_sync();
        // 16 columns at a time go through shared memory (per warp two buffers of 32 rows x 16
        // columns, 64-byte swizzle: 16-byte piece j of row r at piece j ^ ((r >> 1) & 3)).  From
        // there one TMA store (first partial sum) or fp32 add-reduction per buffer moves whole
        // 64-byte row pieces; rows and columns outside the output are clipped by TMA.  O is free
        // for the tensor core again as soon as its last columns have been read.
        const uint32_t stage = flush_stage + (uint32_t)q * 4096;
        if (a.out_tma) {
            if (lane == 0) ptx::bulk_wait<0>();   // the previous flush's reductions are complete (order of the sums)
            __syncwarp();
            // one K split: the output itself, problem = third coordinate; several: the slabs, stacked
            const int y = (a.KS == 1 ? 0 : (prob * a.KS + ks) * a.slab_rows) + m0 + q * 32;
            const int z = a.KS == 1 ? prob : 0;
#pragma unroll 1
            for (int c = 0; c < a.NT / 16; ++c) {
                const uint32_t buf = stage + (uint32_t)(c & 1) * 2048;
                if (c >= 2) {
                    if (lane == 0) ptx::bulk_wait_read<1>();   // the buffer's previous contents have been read
                    __syncwarp();
                }
                uint32_t r[16];
                ptx::tmem_ld_32x16(tmem + lane_addr + Cfg::COL_O + ob * kFusedNT + c * 16, r);
                if (cat_halves) {   // hi * lo part of a 64-column tile (see GEMM2)
                    uint32_t r2[16];
                    ptx::tmem_ld_32x16(tmem + lane_addr + Cfg::COL_O + ob * kFusedNT + 64 + c * 16, r2);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) + __uint_as_float(r2[i]));
                }
                ptx::tmem_ld_wait();
                if (c == a.NT / 16 - 1) {
                    ptx::tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(o_free(ob));
                }
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(buf + (uint32_t)lane * 64 + (uint32_t)((j ^ ((lane >> 1) & 3)) << 4)),
                                 "r"(r[4 * j]), "r"(r[4 * j + 1]), "r"(r[4 * j + 2]), "r"(r[4 * j + 3]) : "memory");
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    if (first_sum) ptx::tma_store_3d(&tm_out, buf, n0 + c * 16, y, z);
                    else ptx::tma_reduce_add_3d(&tm_out, buf, n0 + c * 16, y, z);
                    ptx::bulk_commit();
                }
            }
        } else {
            // output rows that are not 16-byte aligned: the same through plain stores / atomics
            float *obase = a.out + (a.KS == 1 ? prob * a.stride_O : (long long)(prob * a.KS + ks) * a.slab) +
                           (long long)(m0 + q * 32) * a.ld_out;
            const int ncols = a.KS == 1 ? a.N : a.Nt * a.NT;   // slabs are padded to whole tiles
            const int nrows = a.KS == 1 ? a.M : a.M + kFusedRows;   // ... and to whole row tiles
#pragma unroll 1
            for (int c = 0; c < a.NT / 16; ++c) {
                uint32_t r[16];
                ptx::tmem_ld_32x16(tmem + lane_addr + Cfg::COL_O + ob * kFusedNT + c * 16, r);
                if (cat_halves) {
                    uint32_t r2[16];
                    ptx::tmem_ld_32x16(tmem + lane_addr + Cfg::COL_O + ob * kFusedNT + 64 + c * 16, r2);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) + __uint_as_float(r2[i]));
                }
                ptx::tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stage + (uint32_t)lane * 64 + (uint32_t)((j ^ ((lane >> 1) & 3)) << 4)),
                                 "r"(r[4 * j]), "r"(r[4 * j + 1]), "r"(r[4 * j + 2]), "r"(r[4 * j + 3]) : "memory");
                __syncwarp();
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const int rr = t * 8 + (lane >> 2), pc = lane & 3;
                    uint32_t x[4];
                    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(x[0]), "=r"(x[1]), "=r"(x[2]), "=r"(x[3])
                                 : "r"(stage + (uint32_t)rr * 64 + (uint32_t)((pc ^ ((rr >> 1) & 3)) << 4)) : "memory");
                    const int n = n0 + c * 16 + pc * 4;
                    if (m0 + q * 32 + rr < nrows) {
                        float *dst = obase + (long long)rr * a.ld_out + n;
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            if (n + e >= ncols) continue;
                            if (first_sum) dst[e] = __uint_as_float(x[e]);   // the first partial sum initialises the target
                            else atomicAdd(dst + e, __uint_as_float(x[e]));
                        }
                    }
                }
                __syncwarp();
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(o_free(ob));
        }
        return true;
    };

    if (warp == kFusedTmaWarp) {
        // ---------------- TMA producer: per block NCH_B chunks of B rows, then NCH_D chunks of D rows ----------------
        if (lane == 0) {
            if (!SPMM) { ptx::tma_prefetch_desc(&tm_bhi); if (!EXACT) ptx::tma_prefetch_desc(&tm_blo); }
            if (FUSED) { ptx::tma_prefetch_desc(&tm_dhi); if (!EXACT) ptx::tma_prefetch_desc(&tm_dlo); }
            // Chunk order = the order the MMA thread consumes them: B(0); then per block b:
            // D(b,0) D(b,1) | B(b+1) | D(b,2) D(b,3)   (SDDMM: B chunks only; last block of a chunk: B(b+1) last).
            int c = 0;
            // first row of the CTA's block 0 in the stacked operand copies, column tile, and (balanced partition) the
            // block at which the next segment begins
            int seg_col0 = krow0 + b0 * kFusedBlk, ntile = nt, seg_end = bal ? 0 : nblk;
            auto put = [&](bool is_b, int blk, int i) -> bool {
                const int s = c % RING;
                if (c >= RING && !ptx::mbar_wait(empty(s), ((c / RING) - 1) & 1)) return false;
                if (c == a.debug_drop_chunk) { ++c; return true; }   // (test hook: nobody will ever complete this chunk's barrier)
                const uint32_t dst = ring + s * kFusedChunk;
                if (bal && blk >= seg_end) {   // a later segment than the one before (the blocks come in increasing order)
                    const uint32_t sg = seg_at(blk);
                    seg_col0 = seg_f(sg, kSegProb) * a.Kp + (seg_f(sg, kSegBt0) - seg_f(sg, kSegStart)) * kFusedBlk;
                    ntile = seg_f(sg, kSegNt);
                    seg_end = sg + 32 < segtab + 32 * (uint32_t)ptx::lds32(segtab - 8) ? seg_f(sg + 32, kSegStart) : nblk;
                }
                const int col0 = seg_col0 + blk * kFusedBlk;
                ptx::mbar_arrive_expect_tx(full(s), (is_b ? kFusedChunk : 2 * kFusedW * a.NT * 4) / (EXACT ? 2 : 1));   // hi (+ lo)
                if (is_b) {   // B rows col0..col0+127, k group i
                    ptx::tma_load_3d(dst, &tm_bhi, full(s), 0, col0, i);
                    if (!EXACT) ptx::tma_load_3d(dst + kFusedChunk / 2, &tm_blo, full(s), 0, col0, i);
                } else {      // D rows of window i of the block
                    const int krow = col0 + i * kFusedW;
                    ptx::tma_load_3d(dst, &tm_dhi, full(s), 0, krow, ntile * (a.NT / 32));
                    // (64-column O tiles: the lo copy sits right behind the 8 KB hi copy, so that [hi | lo] is one
                    // MN-major operand of 128 columns, see GEMM2)
                    if (!EXACT) ptx::tma_load_3d(dst + (a.NT == 64 ? kFusedW * 64 * 4 : kFusedChunk / 2), &tm_dlo, full(s), 0, krow, ntile * (a.NT / 32));
                }
                ++c;
                return true;
            };
            for (int i = 0; i < NCH_B && nblk > 0 && !failed; ++i) failed = !put(true, 0, i);
            for (int b = 0; b < nblk && !failed; ++b) {
                // (FusedMM: at the end of a chunk of blocks GEMM1 of the next block comes last, see the MMA thread)
                const bool late_b = FUSED && b % kFusedFlushBlocks == kFusedFlushBlocks - 1;
                if (FUSED) for (int w = 0; w < 2 && !failed; ++w) failed = !put(false, b, w);
                if (!SPMM && b + 1 < nblk && !late_b) for (int i = 0; i < NCH_B && !failed; ++i) failed = !put(true, b + 1, i);
                if (FUSED) for (int w = 2; w < WPB && !failed; ++w) failed = !put(false, b, w);
                if (!SPMM && b + 1 < nblk && late_b) for (int i = 0; i < NCH_B && !failed; ++i) failed = !put(true, b + 1, i);
            }
            if (failed)
                for (int j = c > RING ? c - RING : 0; j < c; ++j) ptx::mbar_wait(full(j % RING), (j / RING) & 1);
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            constexpr uint32_t idesc1 = ptx::idesc_tf32(kFusedRows, kFusedBlk, false, false);
            const uint32_t idesc2 = a.NT == 64 ? ptx::idesc_tf32(kFusedRows, 64, false, true) : ptx::idesc_tf32(kFusedRows, kFusedNT, false, true);
            constexpr uint32_t idesc2_cat = ptx::idesc_tf32(kFusedRows, kFusedNT, false, true);
            // 64-column O tiles (N <= 64): a 64-column MMA would leave half of the tensor core's width unused (it takes 46
            // cycles, not 32), so P'_hi is multiplied by [D_hi | D_lo] in ONE 128-column MMA whose two halves land in
            // columns 0-63 and 64-127 of the accumulator, P'_lo by D_hi in a 64-column one: two MMAs per K step instead
            // of three; the flush adds the two halves.
            const bool cat = !EXACT && a.NT == 64;
            int c = 0, ppu = 0;   // chunk counter, P' buffer uses so far
            // balanced partition: the next segment whose A tile GEMM1 will need, and its first block
            int a_seg = 1, a_next = (bal && !SPMM && (int)ptx::lds32(segtab - 8) > 1) ? (int)ptx::lds32(segtab + 32 + kSegStart) : -1;
            auto gemm1 = [&](int b) -> bool {   // P = A_tile * B_block^T over NCH_B chunks
                const int pb = FUSED ? 0 : (b & 1);
                const int puse = FUSED ? b : (b >> 1);
                if (puse > 0 && !ptx::mbar_wait(p_free(pb), (puse - 1) & 1)) return false;   // P drained?
                if (bal && !SPMM && b == a_next) {
                    // first block of a new segment: the processors have put the next row tile of A in place
                    if (!ptx::mbar_wait(a_ready, (a_seg - 1) & 1)) return false;
                    ptx::tc_fence_after_sync();
                    ++a_seg;
                    a_next = a_seg < (int)ptx::lds32(segtab - 8) ? (int)ptx::lds32(segtab + a_seg * 32 + kSegStart) : -1;
                }
                const uint32_t pacc = tmem + Cfg::COL_P + pb * kFusedBlk;
                for (int i = 0; i < NCH_B; ++i, ++c) {
                    const int s = c % RING;
                    if (!ptx::mbar_wait(full(s), (c / RING) & 1)) return false;
                    ptx::tc_fence_after_sync();
                    const uint32_t b_hi = ring + s * kFusedChunk, b_lo = b_hi + kFusedChunk / 2;
#pragma unroll
                    for (int k8 = 0; k8 < 4; ++k8) {
                        const uint64_t dbh = ptx::smem_desc(b_hi + k8 * 32, 16, 1024, ptx::kLayoutSw128);
                        const uint64_t dbl = ptx::smem_desc(b_lo + k8 * 32, 16, 1024, ptx::kLayoutSw128);
                        const uint32_t acol = i * 32 + k8 * 8;
                        ptx::mma_tf32_ts(pacc, tmem + Cfg::COL_AHI + acol, dbh, idesc1, (i | k8) != 0);
                        if (EXACT) continue;   // A and B exact in tf32: no lo terms
                        ptx::mma_tf32_ts(pacc, tmem + Cfg::COL_AHI + acol, dbl, idesc1, 1);
                        if (FUSED) {
                            const uint64_t dal = ptx::smem_desc(alo_smem + i * (kFusedRows * 128) + k8 * 32, 16, 1024, ptx::kLayoutSw128);
                            ptx::mma_tf32_ss(pacc, dal, dbh, idesc1, 1);
                        } else {
                            ptx::mma_tf32_ts(pacc, tmem + Cfg::COL_ALO + acol, dbh, idesc1, 1);
                        }
                    }
                    ptx::mma_commit(empty(s));
                }
                ptx::mma_commit(p_full(pb));
                return true;
            };
            auto gemm2 = [&](int b, int w) -> bool {   // O += P'_window * D_window
                const int s = c % RING, ppb = ppu & 1;
                if (!ptx::mbar_wait(pp_full(ppb), (ppu >> 1) & 1)) return false;
                if (!ptx::mbar_wait(full(s), (c / RING) & 1)) return false;
                ptx::tc_fence_after_sync();
                const uint32_t d_hi = ring + s * kFusedChunk, d_lo = d_hi + kFusedChunk / 2;
                const uint32_t pph = tmem + Cfg::COL_PP + ppb * 64, ppl = pph + 32;
                const uint32_t oacc = tmem + Cfg::COL_O + ((b / kFusedFlushBlocks) % NOB) * kFusedNT;
                // D window: MN-major tf32 (32-byte-atom swizzle): column groups 4 KB apart, 4-row K groups 512 B apart,
                // +1 KB per K step of 8 rows.  (Two copies of the loop: a test inside it costs the issuing thread, whose
                // instruction stream paces the tensor pipe, several percent.)
                const uint32_t first = ((b % kFusedFlushBlocks) | w) != 0;   // 0: this MMA starts a new partial sum
                if (cat) {
#pragma unroll
                    for (int k8 = 0; k8 < kFusedW / 8; ++k8) {
                        const uint64_t ddh = ptx::smem_desc(d_hi + k8 * 1024, kFusedW * 128, 512, ptx::kLayoutSw128Base32);
                        ptx::mma_tf32_ts(oacc, pph + k8 * 8, ddh, idesc2_cat, k8 == 0 ? first : 1u);
                        ptx::mma_tf32_ts(oacc, ppl + k8 * 8, ddh, idesc2, 1);
                    }
                } else {
#pragma unroll
                    for (int k8 = 0; k8 < kFusedW / 8; ++k8) {
                        const uint64_t ddh = ptx::smem_desc(d_hi + k8 * 1024, kFusedW * 128, 512, ptx::kLayoutSw128Base32);
                        const uint64_t ddl = ptx::smem_desc(d_lo + k8 * 1024, kFusedW * 128, 512, ptx::kLayoutSw128Base32);
                        ptx::mma_tf32_ts(oacc, pph + k8 * 8, ddh, idesc2, k8 == 0 ? first : 1u);
                        ptx::mma_tf32_ts(oacc, ppl + k8 * 8, ddh, idesc2, 1);
                        if (!EXACT) ptx::mma_tf32_ts(oacc, pph + k8 * 8, ddl, idesc2, 1);
                    }
                }
                ptx::mma_commit(pp_free(ppb));
                ptx::mma_commit(empty(s));
                ++c;
                ++ppu;
                return true;
            };
            // GEMM1 of block b+1 is issued between the second and third GEMM2 of block b: by then the
            // element-wise warps have read all of P(b), and the tensor pipe has work while they
            // process the last two windows of block b.
            if (!SPMM && nblk > 0 && !gemm1(0)) failed = true;
            for (int b = 0; b < nblk && !failed; ++b) {
                // O restarts from zero every kFusedFlushBlocks blocks, once the processors have taken the
                // previous partial sum out of tensor memory
                if (FUSED && b % kFusedFlushBlocks == 0 && b / kFusedFlushBlocks >= NOB) {
                    const int ch = b / kFusedFlushBlocks;   // chunk ch reuses the accumulator of chunk ch - NOB
                    failed = !ptx::mbar_wait(o_free(ch % NOB), (ch / NOB - 1) & 1);
                }
                // At the end of a chunk GEMM1 of the next block is issued after the chunk's last GEMM2, so that
                // the tensor core works on it while the processors take O out of tensor memory.
                const bool late_b = FUSED && b % kFusedFlushBlocks == kFusedFlushBlocks - 1;
                if (FUSED) for (int w = 0; w < 2 && !failed; ++w) failed = !gemm2(b, w);
                if (!SPMM && b + 1 < nblk && !late_b && !failed) failed = !gemm1(b + 1);
                if (FUSED) for (int w = 2; w < WPB && !failed; ++w) failed = !gemm2(b, w);
                if (FUSED && !failed && (late_b || b == nblk - 1))
                    ptx::mma_commit(o_full((b / kFusedFlushBlocks) % NOB));
                if (!SPMM && b + 1 < nblk && late_b && !failed) failed = !gemm1(b + 1);
            }
        }
    } else if ((warp >= 2 && warp < 6) || (Cfg::PSETS == 2 && warp >= 16)) {
        // ---------------- processor warps (thread = row; TMEM lane quarter q) ----------------
        // FusedMM / SPMM: per window, take the row's stored values (densified and transposed by a
        // helper warp into a shared-memory slot), multiply them into P (or use them as they are for
        // SPMM), split to hi/lo and write P' to tensor memory.
        // SDDMM: per window, copy the row of P into a slot; a helper warp writes the stored entries.
        const int nwin = nblk * WPB;
        constexpr int PSETS = Cfg::PSETS;
        const int pset = warp >= 16 ? 1 : 0;   // which set of processor warps this one belongs to
        // (balanced FusedMM: one round per segment, it_end = first window of the next segment; otherwise a single round)
        int it = FUSED ? pset : 0;
        int it_end = (bal && !SPMM && (int)ptx::lds32(segtab - 8) > 1) ? (int)ptx::lds32(segtab + 32 + kSegStart) * WPB : nwin;
        for (;;) {
        for (; it < it_end; it += FUSED ? PSETS : 1) {
            const int blk = it / WPB, w = it % WPB;
            // FusedMM / SPMM: one item (32 rows) per processor warp and window.  SDDMM: two items of 16 rows,
            // lanes 0-15 and lanes 16-31 each with their own slot.
            const int j = FUSED ? it * 4 + q : it * 8 + 2 * q + (lane >> 4);
            const int s = j % NSLOT, use = j / NSLOT;
            const uint32_t slot = slots + s * Cfg::SLOT_BYTES + (FUSED ? lane : (lane & 15)) * 128;
            if (FUSED) {
                float sv[32];
                {
                    bool ok = ptx::mbar_wait(sl_full(s), use & 1);
                    if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
                }
#pragma unroll
                for (int jj = 0; jj < 8; ++jj) {
                    uint32_t x0, x1, x2, x3;
                    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                                 : "=r"(x0), "=r"(x1), "=r"(x2), "=r"(x3)
                                 : "r"(slot + (uint32_t)((jj ^ (lane & 7)) << 4)) : "memory");
                    sv[4 * jj] = __uint_as_float(x0); sv[4 * jj + 1] = __uint_as_float(x1);
                    sv[4 * jj + 2] = __uint_as_float(x2); sv[4 * jj + 3] = __uint_as_float(x3);
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(sl_empty(s));
                uint32_t p0[16], p1[16];
                if (SPMM) {
#pragma unroll
                    for (int c = 0; c < 16; ++c) { p0[c] = 0x3f800000u; p1[c] = 0x3f800000u; }
                } else {
                    if (w < PSETS) {   // this set's first window of the block
                        bool ok = ptx::mbar_wait(p_full(0), blk & 1);
                        if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
                        ptx::tc_fence_after_sync();
                    }
                    const uint32_t pcol = tmem + lane_addr + Cfg::COL_P + w * kFusedW;
                    ptx::tmem_ld_32x16(pcol, p0);
                    ptx::tmem_ld_32x16(pcol + 16, p1);
                    ptx::tmem_ld_wait();
                    if (w + PSETS >= WPB) {   // this set has read its share of the block: GEMM1 may overwrite P once every set has
                        ptx::tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(p_free(0));
                    }
                }
                const int ppb = it & 1, ppuse = it >> 1;
                if (ppuse > 0) {
                    bool ok = ptx::mbar_wait(pp_free(ppb), (ppuse - 1) & 1);
                    if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
                    ptx::tc_fence_after_sync();
                }
                uint32_t hi[16], lo[16];
                const uint32_t pph = tmem + lane_addr + Cfg::COL_PP + ppb * 64, ppl = pph + 32;
#pragma unroll
                for (int c = 0; c < 16; ++c) ptx::split_tf32_fast(__uint_as_float(p0[c]) * sv[c], hi[c], lo[c]);
                ptx::tmem_st_32x16(pph, hi);
                ptx::tmem_st_32x16(ppl, lo);
#pragma unroll
                for (int c = 0; c < 16; ++c) ptx::split_tf32_fast(__uint_as_float(p1[c]) * sv[16 + c], hi[c], lo[c]);
                ptx::tmem_st_32x16(pph + 16, hi);
                ptx::tmem_st_32x16(ppl + 16, lo);
                ptx::tmem_st_wait();
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(pp_full(ppb));
                // ---- flush: after every kFusedFlushBlocks-th block (and after the last block) the partial O
                // leaves tensor memory: each thread adds its row into the output (or
                // its K split's slab): the first partial sum is stored, the later ones are added with fp32
                // reductions (round to nearest).  A given element is only ever touched by the same lane of this
                // warp, in program order, so the sum is reproducible.
                // SPMM: the flush of a chunk of blocks is done one window late (after P' of the next chunk's
                // first window is ready), so that the tensor core has work again the moment O is free.
                // FusedMM: right away; the tensor core runs GEMM1 of the next block meanwhile.
                const bool chunk_ended = SPMM ? (w == 0 && blk > 0 && blk % kFusedFlushBlocks == 0)
                                              : (w == WPB - 1 && blk % kFusedFlushBlocks == kFusedFlushBlocks - 1);
                if (!Cfg::DEDICATED_FLUSH && (chunk_ended || it == nwin - 1)) {
                    const int chunk = (chunk_ended && SPMM) ? blk / kFusedFlushBlocks - 1 : blk / kFusedFlushBlocks;
                    if (!flush_chunk(chunk)) { failed = true; break; }
                }
            } else {
                const int pb = blk & 1;
                if (w == 0) {
                    bool ok = ptx::mbar_wait(p_full(pb), (blk >> 1) & 1);
                    if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
                    ptx::tc_fence_after_sync();
                }
                uint32_t p0[16], p1[16];
                const uint32_t pcol = tmem + lane_addr + Cfg::COL_P + pb * kFusedBlk + w * kFusedW;
                ptx::tmem_ld_32x16(pcol, p0);
                ptx::tmem_ld_32x16(pcol + 16, p1);
                ptx::tmem_ld_wait();
                if (w == WPB - 1) {
                    ptx::tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(p_free(pb));
                }
                if (use > 0) {
                    bool ok = ptx::mbar_wait(sl_empty(s), (use - 1) & 1);
                    if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
                }
#pragma unroll
                for (int jj = 0; jj < 8; ++jj) {
                    const uint32_t *src = jj < 4 ? &p0[4 * jj] : &p1[4 * (jj - 4)];
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(slot + (uint32_t)((jj ^ (lane & 7)) << 4)),
                                 "r"(src[0]), "r"(src[1]), "r"(src[2]), "r"(src[3]) : "memory");
                }
                __syncwarp();
                if ((lane & 15) == 0) ptx::mbar_arrive(sl_full(s));
            }
        }
        if (failed || it_end >= nwin) break;
        // End of a segment of the balanced partition.  GEMM1 of its last block is complete (both sets have read its
        // result), so the A tile makes way for the next segment's: the first set of processors loads it (the second one
        // is flushing O meanwhile), and GEMM1 of the next block waits for its four warps.
        const uint32_t next = seg_at(it_end / WPB);   // the segment that begins there
        if (pset == 0) {
            reload_a_tile<KDP, MODE, EXACT>(a.A, a.lda, a.stride_A, a.M, a.Kd, tmem, lane_addr, alo_smem, row, seg_f(next, kSegM0), seg_f(next, kSegProb));
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(a_ready);
        }
        it_end = next + 32 < segtab + 32 * (uint32_t)ptx::lds32(segtab - 8) ? seg_f(next + 32, kSegStart) * WPB : nwin;
        }
    } else if (Cfg::DEDICATED_FLUSH && warp >= Cfg::FLUSH_WARP0) {
        // ---------------- flusher warps (SPMM): take every chunk's partial sum out of tensor memory ----------------
        const int nchunks = (nblk + kFusedFlushBlocks - 1) / kFusedFlushBlocks;
        for (int chunk = 0; chunk < nchunks; ++chunk)
            if (!flush_chunk(chunk)) { failed = true; break; }
    } else if (helper_index<FUSED>(warp) >= 0 && helper_index<FUSED>(warp) < NH) {
        // ---------------- helper warps: work items (window, group of rows), round-robin ----------------
        // FusedMM / SPMM: fetch the stored values of the item's 32 rows x 32 columns with lane = column
        // (coalesced), densify (0 where nothing is stored; 1 for stored entries when there are no
        // values) and write them transposed into a slot, from which the processor thread of each row
        // reads its row.  SDDMM (items of 16 rows): prefetch the stored values the same way, then take the
        // P rows the processors left in the slot and write the stored entries, one coalesced run per row.
        const int h = helper_index<FUSED>(warp);
        const uint32_t tab = helper_tabs + h * 256;   // 32 records (position, mask) of the item's rows
        constexpr int IR = Cfg::ITEM_ROWS, IPW = Cfg::IPW;
        const int wbase = b0 * WPB, nitems = nblk * WPB * IPW;
        const unsigned lane_bit = 1u << lane, lt_mask = lane_bit - 1u;
        const bool has_values = a.s_values != nullptr;
        const float *s_values = a.s_values + prob * a.stride_sv;           // this problem's stored values,
        const int2 *win = a.win + (size_t)prob * a.M * a.Wk;               // window table
        float *out_values = a.out + prob * a.stride_O;                     // and (SDDMM) output values
        // (balanced partition: the tile and the first window of the segment that holds the items load_rec is asked
        // for, which come in increasing order; in a batch also the problem's window table and the offset of its stored
        // values, which goes into the records' positions)
        int seg_m0 = m0, seg_w0 = wbase, seg_end = bal ? 0 : nitems, seg_pos0 = 0;
        auto load_rec = [&](int jj) {   // lane = row: window record of one row of item jj
            int2 r = make_int2(0, 0);
            if (bal && jj >= seg_end && jj < nitems) {   // the item is in a later segment than the one before: read its record
                const uint32_t sg = seg_at(jj / (IPW * WPB));
                seg_m0 = seg_f(sg, kSegM0);
                seg_w0 = (seg_f(sg, kSegBt0) - seg_f(sg, kSegStart)) * WPB;
                if (a.batch > 1) {   // the segment's problem: its window table, and where its stored values begin
                    win = a.win + (size_t)seg_f(sg, kSegProb) * a.M * a.Wk;
                    seg_pos0 = seg_f(sg, kSegProb) * (int)a.stride_sv;
                }
                seg_end = sg + 32 < segtab + 32 * (uint32_t)ptx::lds32(segtab - 8) ? seg_f(sg + 32, kSegStart) * (IPW * WPB) : nitems;
            }
            const int hrow = seg_m0 + (jj % IPW) * IR + lane, wglob = seg_w0 + jj / IPW;
            if (jj < nitems && lane < IR && hrow < a.M && wglob < a.Wk) r = __ldg(win + (size_t)hrow * a.Wk + wglob);
            if (bal) r.x += seg_pos0;
            return r;
        };
        // the records of the next two items are in flight while an item is processed
        int2 rec_next = load_rec(h), rec_next2 = load_rec(h + NH);
        for (int j = h; j < nitems; j += NH) {
            const int s = j % NSLOT, use = j / NSLOT;
            const int2 rec = rec_next;
            rec_next = rec_next2;
            rec_next2 = load_rec(j + 2 * NH);
            __syncwarp();   // everyone is done with the previous item's records
            ptx::sts64(tab + lane * 8, (uint32_t)rec.x, (uint32_t)rec.y);
            __syncwarp();
            float vn[IR];
            int idx[FUSED ? 1 : IR];   // SDDMM: CSR position of the lane's entry in each row (-1: nothing stored)
            ptx::for_each_row<IR>([&](auto rc) {
                constexpr int r = decltype(rc)::value;
                uint32_t pos, m;
                ptx::lds64_off<r * 8>(tab, pos, m);
                const bool present = (m & lane_bit) != 0;
                const int at = (int)pos + __popc(m & lt_mask);
                vn[r] = (present && (!FUSED || !has_values)) ? 1.f : 0.f;
                if (present && has_values) vn[r] = __ldg(s_values + at);
                if (!FUSED) idx[r] = present ? at : -1;
            });
            const uint32_t slot = slots + s * Cfg::SLOT_BYTES;
            if (FUSED) {
                if (use > 0) {
                    bool ok = ptx::mbar_wait(sl_empty(s), (use - 1) & 1);
                    if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
                }
                ptx::for_each_row<IR>([&](auto rc) {
                    constexpr int r = decltype(rc)::value;
                    ptx::sts32_off<r * 128>(slot + (uint32_t)((lane << 2) ^ ((r & 7) << 4)), __float_as_uint(vn[r]));
                });
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(sl_full(s));
            } else {
                {
                    bool ok = ptx::mbar_wait(sl_full(s), use & 1);
                    if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
                }
                // all reads of the slot first (independent loads), then the stores
                ptx::for_each_row<IR>([&](auto rc) {
                    constexpr int r = decltype(rc)::value;
                    vn[r] *= __uint_as_float(ptx::lds32_off<r * 128>(slot + (uint32_t)((lane << 2) ^ ((r & 7) << 4))));
                });
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(sl_empty(s));
                ptx::for_each_row<IR>([&](auto rc) {
                    constexpr int r = decltype(rc)::value;
                    if (idx[FUSED ? 0 : r] >= 0) out_values[idx[FUSED ? 0 : r]] = vn[r];
                });
            }
        }
    }
    if (failed) atomicExch(a.status, 1);
    if (FUSED && (Cfg::DEDICATED_FLUSH ? warp >= Cfg::FLUSH_WARP0 : Cfg::PSETS == 2 ? warp >= 16 : (warp >= 2 && warp < 6)) && lane == 0) {   // this warp's TMA stores / reductions have been performed
        ptx::bulk_wait<0>();
        ptx::fence_proxy_async_all();
    }
    // (Several slabs per output tile: the grid launched behind this one adds them into O, see slab_sum.cuh.)
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        ptx::tmem_dealloc(tmem, 512);
    }
}

}  // namespace b2sp
