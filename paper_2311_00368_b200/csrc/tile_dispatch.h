// Internal interface between the C-ABI entry points and the dense-tile (tensor-core) family.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>

#include "../../include/b2sp.h"

namespace b2sp {

// Byte offsets inside the workspace header that both families agree on.
constexpr size_t kWsStatusOffset = 256;      // int: device status word (0 = ok)
constexpr size_t kWsTileFlagsOffset = 320;   // int[..]: flags written by the tile pre-pass
constexpr size_t kWsSignatureOffset = 448;   // int[16]: which CSR arrays the window table was built from
constexpr size_t kWsHeaderBytes = 512;

// Element type of the dense operands A, B, D.
constexpr int kDenseF32 = 0, kDenseBf16 = 1;

// A batch of independent problems of the same sizes handled by one set of launches: `count` problems, the
// caller's arrays of consecutive problems `*` elements apart (rp: row_ptr; nz: col_idx, stored values and
// SDDMM output values; A, B, D, O: the dense operands and the output).  Every problem's row_ptr starts at 0.
struct BatchDesc {
    int count = 1;
    long long rp = 0, nz = 0, A = 0, B = 0, D = 0, O = 0;
};

// Plans for FusedMM / SPMM (fused = true; SPMM passes Kd = 0) and SDDMM (fused = false) on the dense-tile
// family; `base_off` = first byte after the row family's region.  They need Kd <= 128.  Np is the padded
// width of D (fused only).
struct FusedPlan {
    bool feasible = false;
    int Kdp = 0, Nt = 1, Mt = 0, Wk = 0, KS = 1, Np = 0, Kp = 0;
    int NT = 128;   // O columns per CTA: 64 when N <= 64
    int bal_ctas = 0;   // > 0: the balanced partition over this many CTAs (KS = slabs per output tile then)
    size_t off_win = 0, off_bhi = 0, off_blo = 0, off_dhi = 0, off_dlo = 0, off_part = 0;
    size_t bytes = 0;
};
FusedPlan plan_fused_tile(int M, int K, int Kd, int N, long long nnz, size_t base_off, bool fused, int batch = 1);

// Enqueues pre-pass (or the check of a prepared table), operand splits, tile kernel and K-split reduction.
// The tile kernel leaves immediately if the pre-pass found a row whose columns are not strictly increasing
// (flag at kWsTileFlagsOffset).
// mode: 0 = SDDMM, 1 = FusedMM, 2 = SPMM through the FusedMM pipeline (P' = the stored values)
// A, B, D: fp32 (dtype 0) or bfloat16 (dtype 1) -- the latter are exact in tf32, so their lo halves (copies,
// loads, MMAs) are left out.
b2sp_status fused_tile(const FusedPlan &p, bool prepared, int mode, int M, int K, int Kd, int N, long long nnz,
                       const int *row_ptr, const int *col_idx, const float *s_values, const void *A,
                       long long lda, const void *B, long long ldb, const void *D, long long ldd,
                       float *out, long long ldo, void *workspace, cudaStream_t st, int *launches,
                       bool keep_status = false, const BatchDesc &batch = BatchDesc(), int dtype = 0);

// FusedMM with an output wider than two 128-column tiles runs as SDDMM into a scratch C followed by SPMM
// on C (see b2sp_fusedmm): the plans of the two phases and where C sits in the workspace.
struct TwoPhasePlan {
    bool feasible = false;
    FusedPlan sddmm, spmm;
    size_t off_c = 0, bytes = 0;
};
TwoPhasePlan plan_two_phase(int M, int K, int Kd, int N, long long nnz, size_t base_off);

// True when the dense-tile family is expected to beat the row family for these sizes (op = B2SP_OP_*,
// width = N for SPMM, Kd for SDDMM, the smaller of the two for FusedMM).
bool tile_profitable(int op, int M, int K, int width, long long nnz);

// Offset of the window table inside the workspace (the same for every op) and its size.
size_t pattern_table_offset(int M);
size_t pattern_table_bytes(int M, int K, int batch = 1);

// Builds the window table (`prepared` = false) or checks that the workspace holds one for these
// arrays (`prepared` = true; a mismatch raises the device flag that sends the work to the row kernels).
b2sp_status pattern_pass(bool prepared, int M, int K, long long nnz, const int *row_ptr, const int *col_idx,
                         void *workspace, cudaStream_t st, int *launches, const BatchDesc &batch = BatchDesc());

}  // namespace b2sp
