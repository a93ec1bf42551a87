// Host side of the dense-tile family: planning (tile shape, K split, workspace carving), TMA
// tensor maps, launches.
#include "tile_dispatch.h"

#include <cuda.h>

#include <atomic>
#include <mutex>

#include "tile_kernels.cuh"
#include "tile_fused.cuh"

namespace b2sp {

namespace {

constexpr int kSMs = 148;

// 0 = the planner decides; set through b2sp_debug_force_k_splits (tests of the K-split epilogues, tuning).
std::atomic<int> g_forced_k_splits{0};
std::atomic<int> g_forced_partition{0};   // 0: the library chooses; 1: tiles x K splits only; 2: balanced wherever it is legal
// -1 = off; set through b2sp_debug_inject_wait_timeout (the test of the bounded waits).
std::atomic<int> g_drop_chunk{-1};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                   CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);

// cuTensorMapEncodeTiled through the runtime's driver entry point query (no link against libcuda).
EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// Packed fp32 tensor [groups][rows][32] (column-blocked dense operand); box = [gbox][rbox][32].
// `mn_major` selects the 128-byte swizzle in 32-byte units that MN-major tf32 MMA operands need;
// otherwise the ordinary 128-byte swizzle (K-major operands).
bool make_blocked_map(CUtensorMap *tm, const float *base, int rows, int groups, int rbox, int gbox,
                      bool mn_major)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    cuuint64_t dims[3] = {32, (cuuint64_t)rows, (cuuint64_t)groups};
    cuuint64_t strides[2] = {128, (cuuint64_t)rows * 128};
    cuuint32_t box[3] = {32, (cuuint32_t)rbox, (cuuint32_t)gbox};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE,
               mn_major ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// fp32 matrix [rows][cols] with row stride `ld` elements, as the target of the tile kernel's flush:
// boxes of 16 columns x 32 rows, 64-byte swizzle.  Needs a 16-byte aligned base and row stride.
// `count` such matrices `stride` elements apart (a multiple of four) form the third dimension.
bool make_output_map(CUtensorMap *tm, float *base, long long rows, int cols, long long ld, int count, long long stride)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)count};
    cuuint64_t strides[2] = {(cuuint64_t)ld * 4, (cuuint64_t)(count > 1 ? stride : rows * ld) * 4};
    cuuint32_t box[3] = {16, 32, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Raises a kernel's dynamic shared-memory limit once per kernel (TAG) and device instead of on every launch.
template <int TAG>
bool allow_dynamic_smem(const void *kernel, int bytes)
{
    static std::atomic<unsigned long long> done{0};   // one bit per device
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    const unsigned long long bit = 1ull << (dev & 63);
    if (done.load(std::memory_order_acquire) & bit) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
    done.fetch_or(bit, std::memory_order_release);
    return true;
}

// K splits of a tile; `blocks` = 128-column blocks of S.
int pick_split(int base_tiles, int blocks)
{
    if (const int forced = g_forced_k_splits.load(std::memory_order_relaxed)) {   // b2sp_debug_force_k_splits
        if (forced >= 1 && forced <= blocks) return forced;
    }
    // One wave of long-lived CTAs beats several waves of short ones (each CTA pays a prologue, an
    // epilogue and a partial-output slab): take the largest split that still fits one wave, as long
    // as every split keeps a few pipeline steps.
    int ks = 1;
    if (base_tiles < kSMs) {
        ks = kSMs / base_tiles;
        if (ks > blocks / 4) ks = blocks / 4;
        if (ks > 32) ks = 32;
        if (ks < 1) ks = 1;
    }
    return ks;
}

// The balanced partition (see tile_fused.cuh) of `units` row tiles of `blocks` 128-column blocks each, for an output
// of `nt` column tiles: groups of nt CTAs, the granules of all row tiles (4-block flush granules; single blocks for
// SDDMM) dealt evenly to the groups, one CTA per SM.  Returns the number of CTAs (0: the plain partition, tiles x K
// splits, stays) and the slabs a tile needs (= the most groups that share a row tile).
int pick_balanced(long long units, int nt, int blocks, int ks, int mode, int *slabs)
{
    const int forced = g_forced_partition.load(std::memory_order_relaxed);   // b2sp_debug_force_partition
    const int gran = mode == kModeSddmm ? 1 : kFusedFlushBlocks;            // SDDMM accumulates nothing across blocks
    if (forced == 1 || blocks % gran != 0 || nt > kSMs) return 0;
    const long long gpt = blocks / gran, gtot = units * gpt;
    if (gtot >= 0x7fffffffll / kSMs) return 0;   // (the partition's arithmetic is 32-bit)
    const long long groups = gtot < kSMs / nt ? gtot : kSMs / nt;
    const long long gmax = (gtot + groups - 1) / groups;
    if ((gmax + gpt - 2) / gpt + 1 > kFusedMaxSegs) return 0;   // a CTA would touch too many row tiles
    if (forced != 2) {
        // Worth it when the longest CTA gets clearly shorter than in the plain partition (whose CTAs come in waves).
        // A CTA that goes on into the next row tile reloads its A tile (FusedMM, SDDMM: about a block and a half of
        // time).  Measured: the time falls by about 0.6 of what the lengths promise (more CTAs at work slow each other
        // down), and slabs where the plain partition writes straight into O (one K split) cost a few percent.  At 7/8 of
        // the length: 8192^2 x 128 SPMM -7%, FusedMM -3%, SDDMM -3%; x 256 (one K split) SPMM -4%, FusedMM -1%; 4096^2
        // SDDMM (8 -> 7 blocks per CTA) +3%.  At 2/3 (24576 x 8192, 192 row tiles): -27% / -26% / -27%.
        const long long plain2 = 2 * ((units * nt * ks + kSMs - 1) / kSMs * ((blocks + ks - 1) / ks));
        const long long mine2 = 2 * gmax * gran + (mode == kModeSpmm ? 0 : 3);
        // (SPMM on one column tile: slabs where there were none cost more than 1/8 of the length buys -- 16384 x 4096 x 128,
        // cache-warm: +4%)
        const int percent = mode == kModeSddmm || ks > 1 ? 94 : mode == kModeSpmm && nt == 1 ? 86 : 90;
        if (mine2 * 100 > plain2 * percent) return 0;
    }
    int most = 1;
    const Balance balance((int)gtot, (int)groups);
    for (long long u = 0; u < units; ++u) {
        const int n = balance.groups_of_tile((int)(u * gpt), (int)gpt);
        if (n > most) most = n;
    }
    *slabs = most < 2 ? 2 : most;   // (the kernel reads "one slab" as "straight into the output")
    return (int)(groups * nt);
}

}  // namespace

size_t pattern_table_offset(int M)
{
    return align_up(align_up(kWsHeaderBytes + sizeof(int) * (size_t)M, 256), 1024);
}
size_t pattern_table_bytes(int M, int K, int batch)
{
    return sizeof(int2) * (size_t)batch * (size_t)M * (size_t)((K + kTileKC - 1) / kTileKC);
}

namespace {
// What a window table is built from (for a batch, `nnz` is the distance between the problems' col_idx arrays).
PatternSignature make_signature(int M, int K, int Wk, long long nnz, const int *row_ptr, const int *col_idx,
                                const BatchDesc &batch)
{
    return PatternSignature{kPatternMagic, M, K, Wk, nnz, row_ptr, col_idx, batch.count, batch.rp, batch.nz};
}
}  // namespace

b2sp_status pattern_pass(bool prepared, int M, int K, long long nnz, const int *row_ptr, const int *col_idx,
                         void *workspace, cudaStream_t st, int *launches, const BatchDesc &batch)
{
    char *ws = static_cast<char *>(workspace);
    int *flags = reinterpret_cast<int *>(ws + kWsTileFlagsOffset);
    PatternSignature *sig_dev = reinterpret_cast<PatternSignature *>(ws + kWsSignatureOffset);
    const int Wk = (K + kTileKC - 1) / kTileKC;
    const PatternSignature sig = make_signature(M, K, Wk, nnz, row_ptr, col_idx, batch);
    // A prepared table is used as it is: the tile kernel itself compares the signature stored beside
    // the table with these arrays and raises the fallback flag on a mismatch.
    if (prepared) return B2SP_OK;
    if (cudaMemsetAsync(ws, 0, kWsHeaderBytes, st) != cudaSuccess) return B2SP_ERR_CUDA;
    int2 *win = reinterpret_cast<int2 *>(ws + pattern_table_offset(M));
    if (Wk > kMasksMaxWk) return B2SP_ERR_UNSUPPORTED;
    if (!allow_dynamic_smem<-1>(reinterpret_cast<const void *>(tile_masks_kernel), kMasksMaxWk * 4)) return B2SP_ERR_CUDA;
    const long long cap = kSMs * 64, rows_all = (long long)M * batch.count;
    tile_masks_kernel<<<(unsigned)(rows_all < cap ? rows_all : cap), kMasksWarps * 32, (size_t)Wk * 4, st>>>(
        M, K, Wk, nnz, row_ptr, col_idx, win, flags, sig, sig_dev);
    *launches += 1;
    return cudaGetLastError() == cudaSuccess ? B2SP_OK : B2SP_ERR_CUDA;
}

bool tile_profitable(int op, int M, int K, int width, long long nnz)
{
    // Measured on B200: the dense-tile family costs a fixed ~35 us (pattern pre-pass, operand splits,
    // tile prologue) plus ~1.3 us per million cells of S whatever the density, the row family ~22 us
    // plus ~31 us per million stored entries (width 128).  The cross-over density is therefore about
    // 4.5% on large matrices and rises as the matrix shrinks (16% at 2048^2, never at 1024^2).
    // Operands narrower than 64 use half of a 64-wide tile at best while the row kernels lose nothing
    // (sub-warps share a row): measured at width 32 on 1k^2 ... 32k x 8k, the cross-over is about 3.5x
    // higher for SPMM, 2x for SDDMM, 2.5x for FusedMM.  With 74 or more row tiles (no K split) the last
    // wave of CTAs is partly empty (96 tiles: 65% of the SMs; 192 tiles: two waves, 65%), which the tile
    // family pays in full unless the balanced partition applies: the cross-over rises by the waves' efficiency
    // against the usual 86%.
    if (M < 256 || K < 256 || width < 16 || nnz <= 0) return false;
    const double cells = (double)M * (double)K;
    const double density = (double)nnz / cells;
    // (FusedMM's row kernel does the work of two ops per stored entry, its tile kernel shares the expansion of S
    // between them: a fit over the 72 grid cases puts its cross-over lower)
    double crossover = op == B2SP_OP_FUSEDMM ? 0.035 + 0.3e6 / cells : 0.045 + 0.5e6 / cells;
    const int tiles = (M + kFusedRows - 1) / kFusedRows;
    if (tiles >= kSMs / 2 && width <= kFusedNT) {
        const int waves = (tiles + kSMs - 1) / kSMs;
        double eff = (double)tiles / ((double)waves * kSMs);
        // (the balanced partition, where the planner takes it, wins back about 0.6 of what the waves lose)
        int slabs = 0;
        const int blocks = (K + kFusedBlk - 1) / kFusedBlk;
        if (pick_balanced(tiles, 1, blocks, pick_split(tiles, blocks), op == B2SP_OP_SDDMM ? kModeSddmm : op == B2SP_OP_SPMM ? kModeSpmm : kModeFused, &slabs))
            eff += 0.6 * (1.0 - eff);
        const double factor = 0.86 / eff;
        crossover *= factor < 1.0 ? 1.0 : factor > 1.35 ? 1.35 : factor;
    }
    const double narrow = op == B2SP_OP_SPMM ? 3.5 : op == B2SP_OP_SDDMM ? 2.0 : 2.5;
    return density >= (width >= 64 ? crossover : narrow * crossover);
}

FusedPlan plan_fused_tile(int M, int K, int Kd, int N, long long nnz, size_t base_off, bool fused, int batch)
{
    FusedPlan p;
    if (batch < 1 || (long long)batch * ((K + kFusedBlk - 1) / kFusedBlk * kFusedBlk) > 0x7fffff00ll) return p;   // stacked operand rows are int coordinates
    if (M <= 0 || K <= 0 || Kd < 0 || Kd > 128 || nnz <= 0 || (fused && N <= 0) || (!fused && Kd == 0)) return p;
    p.Wk = (K + kFusedW - 1) / kFusedW;
    p.Kp = (K + kFusedBlk - 1) / kFusedBlk * kFusedBlk;   // operand copies padded to whole 128-column blocks
    p.Kdp = Kd == 0 ? 0 : Kd <= 32 ? 32 : Kd <= 64 ? 64 : 128;   // Kd == 0: SPMM through the fused pipeline
    p.Mt = (M + kFusedRows - 1) / kFusedRows;
    p.NT = fused && N <= 64 ? 64 : kFusedNT;   // a 64-column GEMM2 costs 46 instead of 64 cycles per MMA
    p.Nt = fused ? (N + p.NT - 1) / p.NT : 1;
    p.Np = fused ? p.Nt * p.NT : 0;
    size_t win_bytes = sizeof(int2) * (size_t)batch * (size_t)M * (size_t)p.Wk;
    if (win_bytes > (size_t)2 << 30 || p.Wk > kMasksMaxWk) return p;
    p.KS = pick_split(batch * p.Mt * p.Nt, p.Kp / kFusedBlk);
    if ((long long)batch * nnz < 0x7fffffffll) {   // (positions in a batch's stacked values are ints)
        int slabs = 0;
        p.bal_ctas = pick_balanced((long long)batch * p.Mt, p.Nt, p.Kp / kFusedBlk, p.KS, !fused ? kModeSddmm : Kd == 0 ? kModeSpmm : kModeFused, &slabs);
        if (p.bal_ctas) p.KS = fused ? slabs : 1;   // (SDDMM has no partial outputs)
    }
    size_t off = align_up(base_off, 1024);
    p.off_win = off;
    off = align_up(off + win_bytes, 1024);
    size_t bbytes = sizeof(float) * (size_t)batch * (size_t)p.Kp * (size_t)p.Kdp;
    p.off_bhi = off;
    off = align_up(off + bbytes, 1024);
    p.off_blo = off;
    off = align_up(off + bbytes, 1024);
    if (fused) {
        size_t dbytes = sizeof(float) * (size_t)batch * (size_t)p.Kp * (size_t)p.Np;
        p.off_dhi = off;
        off = align_up(off + dbytes, 1024);
        p.off_dlo = off;
        off = align_up(off + dbytes, 1024);
        p.off_part = off;
        if (p.KS > 1) off += sizeof(float) * (size_t)batch * (size_t)p.KS * (size_t)p.Mt * kFusedRows * (size_t)p.Np;
    }
    p.bytes = align_up(off, 256);
    p.feasible = true;
    return p;
}

TwoPhasePlan plan_two_phase(int M, int K, int Kd, int N, long long nnz, size_t base_off)
{
    TwoPhasePlan t;
    t.sddmm = plan_fused_tile(M, K, Kd, 0, nnz, base_off, false);
    t.spmm = plan_fused_tile(M, K, 0, N, nnz, base_off, true);
    if (!t.sddmm.feasible || !t.spmm.feasible) return t;
    t.off_c = align_up(t.sddmm.bytes > t.spmm.bytes ? t.sddmm.bytes : t.spmm.bytes, 256);
    t.bytes = align_up(t.off_c + sizeof(float) * (size_t)nnz, 256);
    t.feasible = true;
    return t;
}

namespace {

template <int KDP, int MODE, int PART, bool EXACT>
b2sp_status launch_fused_tile(const CUtensorMap &bh, const CUtensorMap &bl, const CUtensorMap &dh,
                              const CUtensorMap &dl, const CUtensorMap &out, const FusedTileArgs &a, int items,
                              cudaStream_t st)
{
    using Cfg = FusedCfg<KDP, MODE, EXACT>;
    auto kern = fused_tile_kernel<KDP, MODE, PART, EXACT>;
    if (!allow_dynamic_smem<KDP * 32 + MODE * 8 + PART * 2 + (EXACT ? 1 : 0)>(reinterpret_cast<const void *>(kern), Cfg::SMEM_BYTES)) return B2SP_ERR_CUDA;
    // a programmatic dependent of the operand-split kernel: its CTAs are placed while that kernel still runs
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)items);
    cfg.blockDim = dim3(Cfg::THREADS);
    cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kern, bh, bl, dh, dl, out, a);
    return cudaGetLastError() == cudaSuccess ? B2SP_OK : B2SP_ERR_CUDA;
}

// Picks the instantiation: PART from the plan, EXACT from the operand type, KDP from the padded Kd (SPMM has no A / B:
// only its KDP = 32 instantiation exists).
template <int MODE, int PART, bool EXACT>
b2sp_status launch_fused_part(int kdp, const CUtensorMap &bh, const CUtensorMap &bl, const CUtensorMap &dh, const CUtensorMap &dl,
                              const CUtensorMap &out, const FusedTileArgs &a, int items, cudaStream_t st)
{
    if constexpr (MODE == kModeSpmm) {
        return launch_fused_tile<32, MODE, PART, EXACT>(bh, bl, dh, dl, out, a, items, st);
    } else {
        if (kdp == 32) return launch_fused_tile<32, MODE, PART, EXACT>(bh, bl, dh, dl, out, a, items, st);
        if (kdp == 64) return launch_fused_tile<64, MODE, PART, EXACT>(bh, bl, dh, dl, out, a, items, st);
        return launch_fused_tile<128, MODE, PART, EXACT>(bh, bl, dh, dl, out, a, items, st);
    }
}

template <int MODE>
b2sp_status launch_fused_kdp(int kdp, bool exact, const CUtensorMap &bh, const CUtensorMap &bl, const CUtensorMap &dh,
                             const CUtensorMap &dl, const CUtensorMap &out, const FusedTileArgs &a, int items,
                             cudaStream_t st)
{
    if (a.bal_ctas > 0)
        return exact ? launch_fused_part<MODE, kPartBalanced, true>(kdp, bh, bl, dh, dl, out, a, items, st)
                     : launch_fused_part<MODE, kPartBalanced, false>(kdp, bh, bl, dh, dl, out, a, items, st);
    if constexpr (MODE == kModeFused) {   // (only FusedMM is offered on batches)
        if (a.batch > 1)
            return exact ? launch_fused_part<MODE, kPartBatched, true>(kdp, bh, bl, dh, dl, out, a, items, st)
                         : launch_fused_part<MODE, kPartBatched, false>(kdp, bh, bl, dh, dl, out, a, items, st);
    }
    return exact ? launch_fused_part<MODE, kPartTiles, true>(kdp, bh, bl, dh, dl, out, a, items, st)
                 : launch_fused_part<MODE, kPartTiles, false>(kdp, bh, bl, dh, dl, out, a, items, st);
}

// Splits (or only checks) up to three dense operands and clears the device status word.
void launch_split(const SplitJobs &jobs, int *status, const TableCheck &chk, cudaStream_t st)
{
    long long most = 1;
    for (int i = 0; i < jobs.n; ++i) {
        const long long g = (long long)jobs.j[i].batch * jobs.j[i].rows_p * (jobs.j[i].cols_p >> 2);
        if (g > most) most = g;
    }
    const long long want = (most + 255) / 256, cap = (long long)kSMs * 8;
    dim3 grid((unsigned)(want < cap ? want : cap), (unsigned)jobs.n);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = chk.after_prepass ? attr : nullptr;   // beside the pattern pre-pass of the same call, never beside foreign work
    cfg.numAttrs = chk.after_prepass ? 1 : 0;
    cudaLaunchKernelEx(&cfg, split_dense_kernel, jobs, status, chk);
}

}  // namespace

b2sp_status fused_tile(const FusedPlan &p, bool prepared, int mode, int M, int K, int Kd, int N, long long nnz,
                       const int *row_ptr, const int *col_idx, const float *s_values, const void *A,
                       long long lda, const void *B, long long ldb, const void *D, long long ldd,
                       float *out, long long ldo, void *workspace, cudaStream_t st, int *launches, bool keep_status,
                       const BatchDesc &batch, int dtype)
{
    const int nb = batch.count;
    const bool exact = dtype == kDenseBf16;   // operands exact in tf32: no lo halves anywhere
    char *ws = static_cast<char *>(workspace);
    int *status = reinterpret_cast<int *>(ws + kWsStatusOffset);
    int *flags = reinterpret_cast<int *>(ws + kWsTileFlagsOffset);
    int2 *win = reinterpret_cast<int2 *>(ws + p.off_win);
    float *bhi = reinterpret_cast<float *>(ws + p.off_bhi), *blo = reinterpret_cast<float *>(ws + p.off_blo);
    float *dhi = reinterpret_cast<float *>(ws + p.off_dhi), *dlo = reinterpret_cast<float *>(ws + p.off_dlo);
    float *part = reinterpret_cast<float *>(ws + p.off_part);

    const bool fused = mode != kModeSddmm, spmm = mode == kModeSpmm;
    CUtensorMap tm_bh, tm_bl, tm_dh, tm_dl;
    if (!spmm && (!make_blocked_map(&tm_bh, bhi, nb * p.Kp, p.Kdp / 32, kFusedBlk, 1, false) ||
                  (!exact && !make_blocked_map(&tm_bl, blo, nb * p.Kp, p.Kdp / 32, kFusedBlk, 1, false))))
        return B2SP_ERR_CUDA;
    if (fused) {
        if (!make_blocked_map(&tm_dh, dhi, nb * p.Kp, p.Np / 32, kFusedW, p.NT / 32, true) ||
            (!exact && !make_blocked_map(&tm_dl, dlo, nb * p.Kp, p.Np / 32, kFusedW, p.NT / 32, true)))
            return B2SP_ERR_CUDA;
    } else {
        tm_dh = tm_bh;   // unused by the SDDMM kernel
    }
    if (spmm) tm_bh = tm_dh;   // unused by the SPMM mode
    if (exact || !fused) tm_dl = tm_dh;   // (maps the kernel never touches still have to be valid objects)
    if (exact || spmm) tm_bl = tm_bh;
    {
        b2sp_status prc = pattern_pass(prepared, M, K, nnz, row_ptr, col_idx, workspace, st, launches, batch);
        if (prc != B2SP_OK) return prc;
    }
    {
        // B and D are split into tf32 hi/lo copies; A, which the tile kernel splits itself, is only checked
        // for non-finite values (see split_dense_kernel).
        const int a_rows_p = (M + 3) & ~3, a_cols_p = (Kd + 31) & ~31;
        const SplitJob jb{B, ldb, K, Kd, bhi, exact ? nullptr : blo, p.Kp, p.Kdp, nb, batch.B, dtype, 0};
        const SplitJob jd{D, ldd, K, N, dhi, exact ? nullptr : dlo, p.Kp, p.Np, nb, batch.D, dtype, 0};
        const SplitJob ja{A, lda, M, Kd, nullptr, nullptr, a_rows_p, a_cols_p, nb, batch.A, dtype, 1};
        SplitJobs jobs;
        jobs.n = 0;
        jobs.has_check = 0;
        jobs.check = ja;
        if (!spmm) { jobs.j[jobs.n++] = jb; jobs.has_check = 1; }
        if (fused) jobs.j[jobs.n++] = jd;
        int *clear = keep_status ? nullptr : status;
        // (a prepared table is checked against this call's arrays here, so that the flags are final before the tile kernel)
        const TableCheck chk{make_signature(M, K, p.Wk, nnz, row_ptr, col_idx, batch),
                             prepared ? reinterpret_cast<const PatternSignature *>(ws + kWsSignatureOffset) : nullptr, flags,
                             prepared ? 0 : 1};
        launch_split(jobs, clear, chk, st);
        *launches += 1;
    }
    if (cudaGetLastError() != cudaSuccess) return B2SP_ERR_CUDA;

    FusedTileArgs a;
    a.M = M; a.K = K; a.Kd = Kd; a.Kdp = p.Kdp; a.N = N; a.Wk = p.Wk; a.KS = p.KS; a.Nt = p.Nt; a.NT = p.NT;
    a.batch = nb; a.ctas_per_problem = p.Mt * p.Nt * p.KS; a.Kp = p.Kp;
    a.tiles_pp = p.Mt * p.Nt; a.bal_ctas = p.bal_ctas;
    a.stride_sv = batch.nz; a.stride_A = batch.A; a.stride_O = fused ? batch.O : batch.nz;
    a.win = win; a.s_values = s_values; a.A = A; a.lda = lda;
    a.flags = flags; a.status = status;
    a.debug_drop_chunk = g_drop_chunk.load(std::memory_order_relaxed);
    a.O = out; a.ldo = ldo;
    if (!fused) { a.out = out; a.ld_out = 0; a.slab = 0; }
    else if (p.KS == 1) { a.out = out; a.ld_out = ldo; a.slab = 0; }
    else { a.out = part; a.ld_out = p.Np; a.slab = (long long)p.Mt * kFusedRows * p.Np; }
    // The flush goes through TMA when the target's rows are 16-byte aligned (slabs always are).
    CUtensorMap tm_out = tm_dh;
    a.out_tma = 0;
    a.slab_rows = p.Mt * kFusedRows;
    if (fused) {
        // (TMA clips out-of-range columns in units of 16 bytes: a width that is not a multiple of four
        // would let it write up to three floats past the end of every row of O)
        const bool aligned = (reinterpret_cast<uintptr_t>(a.out) & 15) == 0 && (a.ld_out & 3) == 0 &&
                             (p.KS > 1 || ((N & 3) == 0 && (batch.O & 3) == 0));
        if (aligned) {
            // one K split: the caller's outputs, one per problem along the third dimension; several: the slabs
            // of all problems and splits, stacked along the rows
            const long long rows = p.KS == 1 ? M : (long long)nb * p.KS * a.slab_rows;
            const int cols = p.KS == 1 ? N : p.Np;
            if (!make_output_map(&tm_out, a.out, rows, cols, a.ld_out, p.KS == 1 ? nb : 1, batch.O)) return B2SP_ERR_CUDA;
            a.out_tma = 1;
        }
    }
    const int items = p.bal_ctas ? p.bal_ctas : nb * p.Mt * p.Nt * p.KS;
    b2sp_status rc = spmm    ? launch_fused_kdp<kModeSpmm>(32, exact, tm_bh, tm_bl, tm_dh, tm_dl, tm_out, a, items, st)
                     : fused ? launch_fused_kdp<kModeFused>(p.Kdp, exact, tm_bh, tm_bl, tm_dh, tm_dl, tm_out, a, items, st)
                             : launch_fused_kdp<kModeSddmm>(p.Kdp, exact, tm_bh, tm_bl, tm_dh, tm_dl, tm_out, a, items, st);
    *launches += 1;
    if (rc != B2SP_OK) return rc;
    if (fused && p.KS > 1) {
        // several slabs per output tile: a kernel of its own, behind the tile kernel, adds them into O (slab_sum.cuh)
        SlabSumArgs sa;
        sa.slabs = part; sa.slab = a.slab; sa.ld = p.Np; sa.KS = p.KS;
        sa.O = out; sa.ldo = ldo; sa.stride_O = batch.O;
        sa.M = M; sa.N = N; sa.batch = nb; sa.Mt = p.Mt; sa.Nt = p.Nt; sa.NT = p.NT;
        sa.gpt = p.Kp / kFusedBlk / kFusedFlushBlocks; sa.bal_ctas = p.bal_ctas;
        sa.flags = flags;
        const long long threads = (long long)nb * M * ((N + 3) / 4);
        // (four CTAs per SM: all of them start at once when the tile kernel's CTAs leave, so the gated row kernel, this grid's
        // programmatic dependent, starts beside them and not after a second wave; measured against eight: FusedMM and SPMM -1%)
        const long long want = (threads + 255) / 256, cap = (long long)kSMs * 4;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(want < cap ? want : cap));
        cfg.blockDim = dim3(256);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaLaunchKernelEx(&cfg, slab_sum_kernel, sa);
        *launches += 1;
        if (cudaGetLastError() != cudaSuccess) return B2SP_ERR_CUDA;
    }
    return B2SP_OK;
}

}  // namespace b2sp

// Debug / tuning hook declared in include/b2sp_debug.h.
extern "C" void b2sp_debug_force_k_splits(int k_splits)
{
    b2sp::g_forced_k_splits.store(k_splits > 0 ? k_splits : 0, std::memory_order_relaxed);
}

// Debug / tuning hook declared in include/b2sp_debug.h.
extern "C" void b2sp_debug_force_partition(int partition)
{
    b2sp::g_forced_partition.store(partition == 1 || partition == 2 ? partition : 0, std::memory_order_relaxed);
}

// Debug hook declared in include/b2sp_debug.h.
extern "C" b2sp_status b2sp_debug_inject_wait_timeout(int chunk, unsigned long long limit_ns)
{
    const unsigned long long limit = chunk >= 0 && limit_ns > 0 ? limit_ns : b2sp::ptx::kWaitLimitNs;
    if (cudaMemcpyToSymbol(b2sp::ptx::c_wait_limit_ns, &limit, sizeof(limit)) != cudaSuccess) return B2SP_ERR_CUDA;
    b2sp::g_drop_chunk.store(chunk >= 0 ? chunk : -1, std::memory_order_relaxed);
    return B2SP_OK;
}
