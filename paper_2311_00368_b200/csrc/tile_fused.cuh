// Dense-tile FusedMM and SDDMM (tcgen05 / TMEM / TMA, 3xTF32) over the window table of S.
//
// One CTA owns 128 rows of S (= rows of A and O) and a range of 32-column windows of S.
//   * A_tile (128 x Kd) is split into tf32 hi/lo once and kept in tensor memory for the CTA's life.
//   * Per window: GEMM1  P = A_tile * B_window^T  (128 x 32, A from TMEM, B rows by TMA), into one of
//     two P accumulators in TMEM.
//   * Four warps (thread = row) read P, apply the window's occupancy mask and the stored values
//     (the sampled C of the paper exists only in these registers), split the result into hi/lo and
//     write it back to TMEM as P'.
//   * FusedMM: GEMM2  O += P' * D_window  (A = P' from TMEM, B = D rows by TMA, MN-major), O in TMEM.
//     SDDMM: the masked values are written to out_values instead (coalesced through shared memory).
// The MMA thread issues GEMM1 of window t+1 before GEMM2 of window t, so the tensor pipe works while
// the element-wise stage of window t runs.
//
// TMEM columns (512 allocated): O [0,128)  P0 [128,160)  P1 [160,192)  P'hi [192,224)  P'lo [224,256)
//                               A_hi [256, 256+Kdp)      A_lo [384, 384+Kdp)          (Kdp <= 128)
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx_sm100.cuh"

#ifdef B2SP_TILE_PROFILE
#define B2SP_FPROF_DECL long long fp_t0 = 0, fp_acc[6] = {0, 0, 0, 0, 0, 0};
#define B2SP_FPROF_START fp_t0 = clock64();
#define B2SP_FPROF_STOP(i) { long long t_ = clock64(); fp_acc[i] += t_ - fp_t0; fp_t0 = t_; }
#define B2SP_FPROF_FLUSH(base) { if (lane == 0 && a.prof) { for (int i_ = 0; i_ < 6; ++i_) atomicAdd(a.prof + (base) + i_, (unsigned long long)fp_acc[i_]); } }
#else
#define B2SP_FPROF_DECL
#define B2SP_FPROF_START
#define B2SP_FPROF_STOP(i) {}
#define B2SP_FPROF_FLUSH(base) {}
#endif

namespace b2sp {

constexpr int kFusedRows = 128;     // rows per CTA (UMMA M)
constexpr int kFusedW = 32;         // S columns per stage (one window)
constexpr int kFusedStages = 3;
constexpr int kFusedThreads = 192;  // warp 0: TMA, warp 1: MMA + TMEM, warps 2-5: element-wise / epilogue
constexpr int kFusedNT = 128;       // O columns per CTA (UMMA N of GEMM2)
constexpr uint32_t kColO = 0, kColP = 128, kColPPhi = 192, kColPPlo = 224, kColAhi = 256, kColAlo = 384;

struct FusedTileArgs {
    int M, K, Kd, Kdp, N, Wk, KS, Nt;
    const int2 *win;          // [M][Wk] window records (position, mask)
    const float *s_values;    // NULL = all ones
    const float *A;           // M x Kd
    long long lda;
    float *out;               // FusedMM: O or partial slabs; SDDMM: out_values
    long long ld_out, slab;
    const int *flags;
    int *status;
    unsigned long long *prof;  // optional role timers (profiling builds only)
};

template <int KDP>
struct FusedCfg {
    static constexpr int B_BYTES = kFusedW * KDP * 4;          // B window tile (hi or lo)
    static constexpr int D_BYTES = kFusedW * kFusedNT * 4;     // D window tile (hi or lo): 16 KB
    static constexpr int STAGE_BYTES = 2 * B_BYTES + 2 * D_BYTES;
    static constexpr int STAGE_BYTES_SDDMM = 2 * B_BYTES;
    static constexpr int AUX_BYTES = 256 /*barriers*/ + 4 * 512 /*record tables*/ + 4 * 4096 /*value staging*/;
    static constexpr int SMEM_BYTES = kFusedStages * STAGE_BYTES + 1024 + AUX_BYTES;
};

// FUSED = true: FusedMM (GEMM2 + O epilogue).  FUSED = false: SDDMM (write the sampled values).
template <int KDP, bool FUSED>
__global__ void __launch_bounds__(kFusedThreads, 1)
fused_tile_kernel(const __grid_constant__ CUtensorMap tm_bhi, const __grid_constant__ CUtensorMap tm_blo,
                  const __grid_constant__ CUtensorMap tm_dhi, const __grid_constant__ CUtensorMap tm_dlo,
                  const FusedTileArgs a)
{
    using Cfg = FusedCfg<KDP>;
    constexpr int STAGES = kFusedStages;
    constexpr int STAGE_BYTES = FUSED ? Cfg::STAGE_BYTES : Cfg::STAGE_BYTES_SDDMM;
    if (a.flags[0] != 0) return;  // pattern not usable for tiles: the row kernels take over

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    const uint32_t aux = smem_base + STAGES * STAGE_BYTES;
    auto full = [&](int s) { return aux + 8u * s; };
    auto empty = [&](int s) { return aux + 8u * (STAGES + s); };
    auto p_full = [&](int b) { return aux + 8u * (2 * STAGES + b); };
    auto p_free = [&](int b) { return aux + 8u * (2 * STAGES + 2 + b); };
    const uint32_t pp_full = aux + 8u * (2 * STAGES + 4), pp_free = aux + 8u * (2 * STAGES + 5);
    const uint32_t o_full = aux + 8u * (2 * STAGES + 6);
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem_gen + STAGES * STAGE_BYTES + 8 * (2 * STAGES + 7));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ks = blockIdx.x % a.KS;
    const int tile = blockIdx.x / a.KS;
    const int nt = tile % a.Nt, mt = tile / a.Nt;
    const int w0 = (int)((long long)a.Wk * ks / a.KS), w1 = (int)((long long)a.Wk * (ks + 1) / a.KS);
    const int nwin = w1 - w0;
    const int m0 = mt * kFusedRows, n0 = nt * kFusedNT;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(full(s), 1); ptx::mbar_init(empty(s), 1); }
        for (int b = 0; b < 2; ++b) { ptx::mbar_init(p_full(b), 1); ptx::mbar_init(p_free(b), 4); }
        ptx::mbar_init(pp_full, 4);
        ptx::mbar_init(pp_free, 1);
        ptx::mbar_init(o_full, 1);
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

    // ---- A tile -> TMEM (hi / lo), done by the element-wise warps; thread = row ----
    const int q = warp & 3;                 // TMEM lane quarter of warps 2..5
    const int row = q * 32 + lane;          // row inside the tile (warps >= 2)
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    if (warp >= 2) {
        const int grow = m0 + row;
        const float *arow = a.A + (long long)(grow < a.M ? grow : 0) * a.lda;
        const bool vec = (a.lda & 3) == 0 && (reinterpret_cast<uintptr_t>(a.A) & 15) == 0;
#pragma unroll 1
        for (int c = 0; c < KDP; c += 16) {
            uint32_t hi[16], lo[16];
            float v[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = 0.f;
            if (grow < a.M) {
                if (vec && c + 16 <= a.Kd) {
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
#pragma unroll
            for (int i = 0; i < 16; ++i) ptx::split_tf32_fast(v[i], hi[i], lo[i]);
            ptx::tmem_st_32x16(tmem + lane_addr + kColAhi + c, hi);
            ptx::tmem_st_32x16(tmem + lane_addr + kColAlo + c, lo);
        }
        ptx::tmem_st_wait();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            ptx::tma_prefetch_desc(&tm_bhi);
            ptx::tma_prefetch_desc(&tm_blo);
            if (FUSED) { ptx::tma_prefetch_desc(&tm_dhi); ptx::tma_prefetch_desc(&tm_dlo); }
            int issued = 0;
            for (int it = 0; it < nwin; ++it) {
                const int s = it % STAGES;
                if (it >= STAGES && !ptx::mbar_wait(empty(s), ((it / STAGES) - 1) & 1)) { failed = true; break; }
                const uint32_t dst = smem_base + s * STAGE_BYTES;
                ptx::mbar_arrive_expect_tx(full(s), STAGE_BYTES);
                const int krow = (w0 + it) * kFusedW;
                ptx::tma_load_3d(dst, &tm_bhi, full(s), 0, krow, 0);
                ptx::tma_load_3d(dst + Cfg::B_BYTES, &tm_blo, full(s), 0, krow, 0);
                if (FUSED) {
                    ptx::tma_load_3d(dst + 2 * Cfg::B_BYTES, &tm_dhi, full(s), 0, krow, nt * (kFusedNT / 32));
                    ptx::tma_load_3d(dst + 2 * Cfg::B_BYTES + Cfg::D_BYTES, &tm_dlo, full(s), 0, krow, nt * (kFusedNT / 32));
                }
                issued = it + 1;
            }
            if (failed)
                for (int it = issued > STAGES ? issued - STAGES : 0; it < issued; ++it)
                    ptx::mbar_wait(full(it % STAGES), (it / STAGES) & 1);
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            constexpr uint32_t idesc1 = ptx::idesc_tf32(kFusedRows, kFusedW, false, false);
            constexpr uint32_t idesc2 = ptx::idesc_tf32(kFusedRows, kFusedNT, false, true);
            B2SP_FPROF_DECL
            B2SP_FPROF_START
            auto gemm1 = [&](int it) -> bool {   // P[it & 1] = A_tile * B_window^T
                const int s = it % STAGES, pb = it & 1;
                if (!ptx::mbar_wait(full(s), (it / STAGES) & 1)) return false;
                B2SP_FPROF_STOP(0)
                if (it >= 2 && !ptx::mbar_wait(p_free(pb), ((it >> 1) - 1) & 1)) return false;
                B2SP_FPROF_STOP(1)
                ptx::tc_fence_after_sync();
                const uint32_t b_hi = smem_base + s * STAGE_BYTES, b_lo = b_hi + Cfg::B_BYTES;
                const uint32_t pacc = tmem + kColP + pb * kFusedW;
#pragma unroll
                for (int kk = 0; kk < KDP / 8; ++kk) {
                    // B window: K-major, one 4 KB sub-tile (32 rows x 128 B, 128-byte swizzle) per 32 k
                    const uint32_t off = (kk >> 2) * (kFusedW * 128) + (kk & 3) * 32;
                    const uint64_t dbh = ptx::smem_desc(b_hi + off, 16, 1024, ptx::kLayoutSw128);
                    const uint64_t dbl = ptx::smem_desc(b_lo + off, 16, 1024, ptx::kLayoutSw128);
                    ptx::mma_tf32_ts(pacc, tmem + kColAhi + kk * 8, dbh, idesc1, kk != 0);
                    ptx::mma_tf32_ts(pacc, tmem + kColAlo + kk * 8, dbh, idesc1, 1);
                    ptx::mma_tf32_ts(pacc, tmem + kColAhi + kk * 8, dbl, idesc1, 1);
                }
                ptx::mma_commit(p_full(pb));
                if (!FUSED) ptx::mma_commit(empty(s));   // SDDMM: the stage only held B
                B2SP_FPROF_STOP(2)
                return true;
            };
            if (nwin > 0 && !gemm1(0)) failed = true;
            for (int it = 0; it < nwin && !failed; ++it) {
                if (it + 1 < nwin && !gemm1(it + 1)) { failed = true; break; }
                if (FUSED) {
                    const int s = it % STAGES;
                    if (!ptx::mbar_wait(pp_full, it & 1)) { failed = true; break; }
                    B2SP_FPROF_STOP(3)
                    ptx::tc_fence_after_sync();
                    const uint32_t d_hi = smem_base + s * STAGE_BYTES + 2 * Cfg::B_BYTES, d_lo = d_hi + Cfg::D_BYTES;
#pragma unroll
                    for (int k8 = 0; k8 < kFusedW / 8; ++k8) {
                        // D window: MN-major tf32 (32-byte-atom swizzle): column groups 4 KB apart, 4-row K
                        // groups 512 B apart, +1 KB per K step of 8 rows
                        const uint64_t ddh = ptx::smem_desc(d_hi + k8 * 1024, kFusedW * 128, 512, ptx::kLayoutSw128Base32);
                        const uint64_t ddl = ptx::smem_desc(d_lo + k8 * 1024, kFusedW * 128, 512, ptx::kLayoutSw128Base32);
                        ptx::mma_tf32_ts(tmem + kColO, tmem + kColPPhi + k8 * 8, ddh, idesc2, (it | k8) != 0);
                        ptx::mma_tf32_ts(tmem + kColO, tmem + kColPPlo + k8 * 8, ddh, idesc2, 1);
                        ptx::mma_tf32_ts(tmem + kColO, tmem + kColPPhi + k8 * 8, ddl, idesc2, 1);
                    }
                    ptx::mma_commit(pp_free);
                    ptx::mma_commit(empty(s));
                    B2SP_FPROF_STOP(4)
                }
            }
            B2SP_FPROF_FLUSH(0)
            if (FUSED && !failed) ptx::mma_commit(o_full);
        }
    } else {
        // ---------------- element-wise warps (thread = row) ----------------
        // Software pipeline over windows: while window t is processed, the stored values of window
        // t+1 are already in flight (loaded cooperatively with lane = column, then transposed through
        // shared memory so that each thread gets its own row), and the record of window t+2 is loading.
        const int ew = warp - 2;
        const uint32_t rec_tab = aux + 256 + ew * 512;              // 2 x 32 records of this warp's rows
        const uint32_t stage_v = aux + 256 + 4 * 512 + ew * 4096;   // 32 x 32 floats, swizzled chunks
        const int grow = m0 + row;
        const int2 *my_win = a.win + (size_t)(grow < a.M ? grow : 0) * a.Wk + w0;
        const unsigned lane_bit = 1u << lane, lt_mask = lane_bit - 1u;
        const bool has_values = a.s_values != nullptr;
        const bool use_tab = has_values || !FUSED;
        auto load_rec = [&](int t) {
            int2 r = make_int2(0, 0);
            if (grow < a.M && t < nwin) r = __ldg(my_win + t);
            return r;
        };
        // column-owner loads of one window's stored values (lane = column, register r = row r of the warp)
        auto issue_values = [&](uint32_t tab, float (&vn)[32]) {
            ptx::for_each_row<32>([&](auto rc) {
                constexpr int r = decltype(rc)::value;
                uint32_t pos, m;
                ptx::lds64_off<r * 8>(tab, pos, m);
                vn[r] = 0.f;
                if (m & lane_bit) vn[r] = __ldg(a.s_values + (pos + __popc(m & lt_mask)));
            });
        };
        // transpose through shared memory: afterwards sv[c] = value of (this thread's row, column c)
        auto transpose_values = [&](const float (&vn)[32], float (&sv)[32]) {
            __syncwarp();
            ptx::for_each_row<32>([&](auto rc) {
                constexpr int r = decltype(rc)::value;
                ptx::sts32_off<r * 128>(stage_v + (uint32_t)((lane << 2) ^ ((r & 7) << 4)), __float_as_uint(vn[r]));
            });
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                uint32_t x0, x1, x2, x3;
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(x0), "=r"(x1), "=r"(x2), "=r"(x3)
                             : "r"(stage_v + lane * 128 + (uint32_t)((j ^ (lane & 7)) << 4)));
                sv[4 * j] = __uint_as_float(x0); sv[4 * j + 1] = __uint_as_float(x1);
                sv[4 * j + 2] = __uint_as_float(x2); sv[4 * j + 3] = __uint_as_float(x3);
            }
        };
        float sv[32], vn[32];
        int2 cur = load_rec(0), nxt = load_rec(1);
        if (use_tab) {
            ptx::sts64(rec_tab + lane * 8, (uint32_t)cur.x, (uint32_t)cur.y);
            __syncwarp();
        }
        if (has_values) {
            issue_values(rec_tab, vn);
            transpose_values(vn, sv);
        }
        B2SP_FPROF_DECL
        B2SP_FPROF_START
        for (int it = 0; it < nwin; ++it) {
            const int pb = it & 1;
            const uint32_t tab_cur = rec_tab + (it & 1) * 256, tab_nxt = rec_tab + ((it + 1) & 1) * 256;
            const unsigned mask = (unsigned)cur.y;
            if (use_tab) {   // records of window it+1 for the whole warp; its values start loading now
                ptx::sts64(tab_nxt + lane * 8, (uint32_t)nxt.x, (uint32_t)nxt.y);
                __syncwarp();
            }
            if (has_values && it + 1 < nwin) issue_values(tab_nxt, vn);
            const int2 nxt2 = load_rec(it + 2);
            if (!has_values) {
#pragma unroll
                for (int c = 0; c < 32; ++c) sv[c] = (mask >> c) & 1u ? 1.f : 0.f;
            }
            B2SP_FPROF_STOP(0)
            {   // P is ready?
                bool ok = ptx::mbar_wait(p_full(pb), (it >> 1) & 1);
                if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
            }
            B2SP_FPROF_STOP(1)
            ptx::tc_fence_after_sync();
            uint32_t p0[16], p1[16];
            ptx::tmem_ld_32x16(tmem + lane_addr + kColP + pb * kFusedW, p0);
            ptx::tmem_ld_32x16(tmem + lane_addr + kColP + pb * kFusedW + 16, p1);
            ptx::tmem_ld_wait();
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(p_free(pb));
            B2SP_FPROF_STOP(2)

            if (FUSED) {
                uint32_t hi[16], lo[16];
                if (it > 0) {
                    bool ok = ptx::mbar_wait(pp_free, (it - 1) & 1);
                    if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
                    ptx::tc_fence_after_sync();
                }
                B2SP_FPROF_STOP(3)
#pragma unroll
                for (int c = 0; c < 16; ++c) ptx::split_tf32_fast(__uint_as_float(p0[c]) * sv[c], hi[c], lo[c]);
                ptx::tmem_st_32x16(tmem + lane_addr + kColPPhi, hi);
                ptx::tmem_st_32x16(tmem + lane_addr + kColPPlo, lo);
#pragma unroll
                for (int c = 0; c < 16; ++c) ptx::split_tf32_fast(__uint_as_float(p1[c]) * sv[16 + c], hi[c], lo[c]);
                ptx::tmem_st_32x16(tmem + lane_addr + kColPPhi + 16, hi);
                ptx::tmem_st_32x16(tmem + lane_addr + kColPPlo + 16, lo);
                ptx::tmem_st_wait();
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(pp_full);
                B2SP_FPROF_STOP(4)
            } else {
                // SDDMM: stage the masked, scaled row (dense, 32 columns) and write the stored entries
                // row by row with lane = column, so each row's outputs are one contiguous store.
                __syncwarp();
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    uint32_t x[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int c = 4 * j + i;
                        x[i] = __float_as_uint(__uint_as_float(c < 16 ? p0[c] : p1[c - 16]) * sv[c]);
                    }
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stage_v + lane * 128 + (uint32_t)((j ^ (lane & 7)) << 4)),
                                 "r"(x[0]), "r"(x[1]), "r"(x[2]), "r"(x[3]) : "memory");
                }
                __syncwarp();
                ptx::for_each_row<32>([&](auto rc) {
                    constexpr int r = decltype(rc)::value;
                    uint32_t pos, m, v;
                    ptx::lds64_off<r * 8>(tab_cur, pos, m);
                    asm volatile("ld.shared.b32 %0, [%1 + %2];" : "=r"(v) : "r"(stage_v + (uint32_t)((lane << 2) ^ ((r & 7) << 4))), "n"(r * 128));
                    if (m & lane_bit) a.out[pos + __popc(m & lt_mask)] = __uint_as_float(v);
                });
            }
            // the values of window it+1 have had the whole step to arrive: give each thread its row
            if (has_values && it + 1 < nwin) transpose_values(vn, sv);
            cur = nxt;
            nxt = nxt2;
        }
        if (ew == 0) { B2SP_FPROF_FLUSH(8) }
        // ---------------- epilogue: O accumulator -> global ----------------
        if (FUSED) {
            {
                bool ok = !failed && ptx::mbar_wait(o_full, 0);
                failed = !__all_sync(0xffffffffu, ok);
            }
            if (!failed) {
                ptx::tc_fence_after_sync();
                float *orow = a.out + (long long)ks * a.slab + (long long)grow * a.ld_out;
                const bool vec = (a.ld_out & 3) == 0 && (reinterpret_cast<uintptr_t>(a.out) & 15) == 0;
#pragma unroll 1
                for (int c = 0; c < kFusedNT / 32; ++c) {
                    uint32_t r[32];
                    ptx::tmem_ld_32x32(tmem + lane_addr + kColO + c * 32, r);
                    ptx::tmem_ld_wait();
                    if (grow < a.M) {
                        const int n = n0 + c * 32;
                        if (vec && n + 32 <= a.N) {
#pragma unroll
                            for (int i = 0; i < 32; i += 4)
                                *reinterpret_cast<uint4 *>(orow + n + i) = make_uint4(r[i], r[i + 1], r[i + 2], r[i + 3]);
                        } else {
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                if (n + i < a.N) orow[n + i] = __uint_as_float(r[i]);
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
        ptx::tmem_dealloc(tmem, 512);
    }
}

}  // namespace b2sp
