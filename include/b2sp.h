/*
 * b2sp -- SPMM, SDDMM and FusedMM over a CSR sparsity pattern S on NVIDIA B200 (sm_100a).
 *
 * C ABI.  Plain pointers and sizes only; `stream` is a cudaStream_t passed as void*
 * (NULL = the legacy default stream).
 *
 * Storage (paper, section "Matrix Storage Layout", Fig. 1):
 *   S  is M x K in compressed sparse row form: row_ptr[M+1], col_idx[nnz], values[nnz];
 *      int32, 0-based; row i owns positions row_ptr[i] <= p < row_ptr[i+1].  Any valid CSR is
 *      accepted: rows may be empty, and the column indices of a row need be neither sorted
 *      nor unique (each stored entry is its own term and its own SDDMM output slot).
 *   Dense operands are fp32, row-major, with a leading dimension counted in elements
 *      (ld >= number of columns).
 *   Names: the paper's (A, I_A; C; B; D; E) are here (S; A; B; D; O); its single letter N is
 *      split into Kd (length of the sampled dot product) and N (width of D and O).
 *
 * Conventions for the device entry points (b2sp_spmm, b2sp_sddmm, b2sp_fusedmm):
 *   - every data pointer is a DEVICE pointer on the current device; the caller owns all of
 *     them, including the workspace; the library allocates nothing;
 *   - inputs are read-only; outputs are fully overwritten (never accumulated into; an empty
 *     row gives a zero output row, Alg. 2 line 1);
 *   - the call enqueues kernels on `stream` and returns without synchronising; it may be captured
 *     into a CUDA graph (make one ordinary call first: it does the library's one-time driver queries);
 *   - `workspace` is scratch of at least b2sp_workspace_bytes(...) bytes, 256-byte aligned;
 *     its contents are overwritten by every call, so two calls that may overlap in time on
 *     the GPU (different streams) need different workspaces;
 *   - argument errors are reported synchronously with no kernel launched; a launch failure
 *     is reported as B2SP_ERR_CUDA; nothing traps, asserts or exits.
 *   - M = 0, nnz = 0 and zero widths are valid (outputs of the stated size are zero-filled).
 *
 * `algo` selects the kernel family:
 *   B2SP_ALGO_AUTO     the library chooses (fastest family whose preconditions hold);
 *   B2SP_ALGO_ROW      CUDA-core row kernels, rows taken longest-first (binned by length);
 *   B2SP_ALGO_ROW_NAT  the same kernels, rows in natural order (no binning pass);
 *   B2SP_ALGO_TILE     dense-tile tensor-core kernels (tcgen05 + tensor memory, every operand
 *                      split into two tf32 numbers so that fp32 accuracy is kept).  A pre-pass
 *                      over col_idx builds a table of 32-column windows; it also detects rows
 *                      whose columns are not strictly increasing, in which case the row kernels
 *                      produce the result instead (decided on the device, inside the same call).
 *                      B2SP_ERR_UNSUPPORTED if the sizes are outside the family (SDDMM/FusedMM:
 *                      Kd > 128), B2SP_ERR_WORKSPACE if the workspace is too small for it.
 *   B2SP_ALGO_TILE_PREPARED  as TILE, but the window table is taken from the workspace, where an
 *                      earlier b2sp_prepare_pattern call for the same S left it (see there).
 * Floating-point results of the families differ in summation order only; all stay within
 * |x - exact| <= 1e-5 * sum|terms| + 1e-6.
 *
 * Non-finite inputs.  The row kernels touch exactly the entries Eq. 1-3 name and follow IEEE
 * propagation.  The dense-tile kernels multiply whole windows of S, positions without a stored entry
 * included (by zero), so they only run when every element of A, B and D -- referenced by a stored
 * entry or not -- is finite and small enough for its tf32 hi part to be finite (|x| below about
 * 3.4e38 * (1 - 2^-11)): the operand pre-pass of every call checks this on the device, and otherwise
 * the row kernels produce that call's result (the check is per call and costs no extra launch).
 * Not checked, and undefined (NaN or Inf) on the dense-tile kernels: stored values s_p that are not
 * finite, and inputs so large that a dot product A_i . B_j overflows fp32 at ANY position (i, j) of
 * S, stored or not (the dense-tile kernels form all of them).
 */
#ifndef B2SP_H
#define B2SP_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    B2SP_OK = 0,
    B2SP_ERR_INVALID_ARG = 1, /* negative size, NULL required pointer, ld < width, nnz > 2^31-1 */
    B2SP_ERR_UNSUPPORTED = 2, /* explicit algo whose preconditions do not hold */
    B2SP_ERR_BAD_CSR = 3,     /* b2sp_validate_csr: row_ptr not monotone / col_idx out of range */
    B2SP_ERR_CUDA = 4,        /* a CUDA runtime call or a kernel launch failed */
    B2SP_ERR_WORKSPACE = 5,   /* workspace NULL, misaligned or too small */
    B2SP_ERR_TIMEOUT = 6,     /* a bounded device-side wait expired (reported by b2sp_device_status) */
    B2SP_ERR_TOO_LARGE = 7    /* the problem does not fit the library's built-in scratch array */
} b2sp_status;

enum { B2SP_ALGO_AUTO = 0, B2SP_ALGO_ROW = 1, B2SP_ALGO_ROW_NAT = 2, B2SP_ALGO_TILE = 3,
       B2SP_ALGO_TILE_PREPARED = 4 };
enum { B2SP_OP_SPMM = 0, B2SP_OP_SDDMM = 1, B2SP_OP_FUSEDMM = 2 };

/* Library version (major*10000 + minor*100 + patch). */
int b2sp_version(void);

/* Static, human-readable name of a status code. */
const char *b2sp_status_string(b2sp_status s);

/*
 * Bytes of device workspace an op needs for the given sizes: an upper bound over all algo values
 * the sizes allow (always a multiple of 256, never 0).  `op` is one of B2SP_OP_*.  Unused sizes
 * (Kd for SPMM, N for SDDMM) may be 0.  Returns 0 on invalid arguments.
 */
size_t b2sp_workspace_bytes(int op, int M, int K, int Kd, int N, long long nnz);

/*
 * The same for one algo value: B2SP_ALGO_AUTO gives what the automatic choice will use (the row
 * family's few bytes per row when it would not pick the dense-tile family), B2SP_ALGO_ROW /
 * B2SP_ALGO_ROW_NAT the row family's size, B2SP_ALGO_TILE / B2SP_ALGO_TILE_PREPARED the dense-tile
 * family's (0 if these sizes are outside that family).  Returns 0 on invalid arguments.
 */
size_t b2sp_workspace_bytes_algo(int op, int algo, int M, int K, int Kd, int N, long long nnz);

/*
 * Pattern analysis shared by the dense-tile kernels of all three ops (work assignment and index
 * staging: where the paper's kernels cut each row's ja array into blocks of VLC = 32 entries on the
 * fly, this library cuts each row into windows of 32 columns once).  Builds, in `workspace`, the
 * table of (first position, occupancy mask) per row and window from row_ptr / col_idx and records
 * which arrays it was built from.  Any later b2sp_spmm / b2sp_sddmm / b2sp_fusedmm call with
 * algo = B2SP_ALGO_TILE_PREPARED, the same workspace and the same M, K, nnz, row_ptr, col_idx
 * skips its own pre-pass.  The caller promises that the contents of row_ptr and col_idx did not
 * change in between; a workspace that does not hold a matching table (never prepared, prepared for
 * another S, or used by a B2SP_ALGO_ROW call since) is detected on the device and the row kernels
 * produce the result instead.  `workspace` must be at least as large as b2sp_workspace_bytes says
 * for the ops that will use it.  Asynchronous on `stream`.
 */
b2sp_status b2sp_prepare_pattern(int M, int K, long long nnz, const int *row_ptr, const int *col_idx,
                                 void *workspace, size_t workspace_bytes, void *stream);

/*
 * SPMM, Eq. 2 / Alg. 2 (SPMM-ROW):  O[i, :] = sum over stored entries (s, k) of row i of
 * s * D[k, :].
 *   M, K, N     S is M x K, D is K x N, O is M x N
 *   nnz         number of stored entries (= row_ptr[M])
 *   row_ptr, col_idx, values   CSR of S (device, read-only)
 *   D, ldd      dense K x N (device, read-only), leading dimension >= N
 *   O, ldo      dense M x N (device, written), leading dimension >= N; must not alias an input
 */
b2sp_status b2sp_spmm(int M, int K, int N, long long nnz,
                      const int *row_ptr, const int *col_idx, const float *values,
                      const float *D, long long ldd, float *O, long long ldo,
                      void *workspace, size_t workspace_bytes, int algo, void *stream);

/*
 * SDDMM, Eq. 1 / Alg. 1 (SDDMM-ROW), with the sampled value scaled by the stored one:
 *   out_values[p] = s_p * sum_{l < Kd} A[i, l] * B[j, l]   for the p-th stored entry (i, j).
 * The paper samples with an all-ones pattern; pass s_values = NULL for that (s_p = 1).
 * The result's sparsity pattern is S's: row_ptr and col_idx are not modified and out_values
 * follows the order of col_idx.
 *   A, lda      dense M x Kd (device, read-only);  B, ldb  dense K x Kd (device, read-only)
 *   out_values  nnz floats (device, written); may be the same pointer as s_values
 *               (in-place, as the paper overwrites its avalues array)
 */
b2sp_status b2sp_sddmm(int M, int K, int Kd, long long nnz,
                       const int *row_ptr, const int *col_idx, const float *s_values,
                       const float *A, long long lda, const float *B, long long ldb,
                       float *out_values,
                       void *workspace, size_t workspace_bytes, int algo, void *stream);

/*
 * FusedMM, Eq. 3 / Alg. 3 (FusedMM-ROW):  O = (S .* (A * B^T)) * D, i.e. the SDDMM values of a
 * row are consumed by the SPMM sweep of the same row without being written to global memory.
 * (One exception, a measured trade: the dense-tile family recomputes the sampled values once per
 * 128-column tile of O, so with N > 256 -- and with 128 < N <= 256 when Kd > 64 and S has at least
 * 3e7 cells -- it writes them once into the workspace and runs its SPMM stage on them, inside the same
 * call.)  s_values may be NULL (all ones).  Arguments as in the two ops above.
 */
b2sp_status b2sp_fusedmm(int M, int K, int Kd, int N, long long nnz,
                         const int *row_ptr, const int *col_idx, const float *s_values,
                         const float *A, long long lda, const float *B, long long ldb,
                         const float *D, long long ldd, float *O, long long ldo,
                         void *workspace, size_t workspace_bytes, int algo, void *stream);

/*
 * The three ops with bfloat16 dense operands and fp32 accumulation -- the variant the paper's conclusion
 * names as its next step.  A, B and D are bfloat16 (the upper 16 bits of an fp32 value; pointers passed as
 * const void*, leading dimensions in elements); the stored values of S, all sums and the outputs stay fp32.
 * Everything else (CSR conventions, workspace from b2sp_workspace_bytes, algo, prepared pattern tables,
 * stream, error behaviour) is as for the fp32 entry points above.  Results satisfy the same bound against
 * Eq. 1-3 evaluated exactly on the bfloat16 values: every product of two bfloat16 numbers is exact in
 * fp32, only the order of the fp32 sums differs.  The row kernels gather half the bytes per dense row;
 * the dense-tile kernels need no lo halves for operands that are exact in tf32, i.e. one tensor-core
 * product per GEMM1 term instead of three and two per GEMM2 term.  The four-element loads of the vector
 * kernels want 8-byte aligned operands and leading dimensions that are multiples of 4 (16 bytes and
 * multiples of 8 for A on the dense-tile kernels); other shapes take the scalar paths.
 */
b2sp_status b2sp_spmm_bf16(int M, int K, int N, long long nnz,
                           const int *row_ptr, const int *col_idx, const float *values,
                           const void *D, long long ldd, float *O, long long ldo,
                           void *workspace, size_t workspace_bytes, int algo, void *stream);
b2sp_status b2sp_sddmm_bf16(int M, int K, int Kd, long long nnz,
                            const int *row_ptr, const int *col_idx, const float *s_values,
                            const void *A, long long lda, const void *B, long long ldb,
                            float *out_values,
                            void *workspace, size_t workspace_bytes, int algo, void *stream);
b2sp_status b2sp_fusedmm_bf16(int M, int K, int Kd, int N, long long nnz,
                              const int *row_ptr, const int *col_idx, const float *s_values,
                              const void *A, long long lda, const void *B, long long ldb,
                              const void *D, long long ldd, float *O, long long ldo,
                              void *workspace, size_t workspace_bytes, int algo, void *stream);

/*
 * FusedMM (Eq. 3 / Alg. 3) on a batch of independent problems of the same sizes in one call -- the rows
 * of Alg. 3 are independent work units, and so are whole problems: e.g. the (batch x heads) problems of
 * sparse attention, O_b = (S_b .* (Q_b * K_b^T)) * V_b.  One pattern pre-pass, one operand pre-pass and one
 * kernel launch cover all problems (CTAs of all problems are in flight together).
 *   batch            number of problems (>= 1)
 *   M, K, Kd, N      sizes of every problem, as for b2sp_fusedmm
 *   row_ptr, row_ptr_stride   problem b's row pointers are row_ptr + b * row_ptr_stride (M + 1 of them,
 *                    starting at 0: positions count inside the problem's own col_idx array);
 *                    row_ptr_stride >= M + 1, or 0 when all problems share one pattern
 *   col_idx, s_values, nnz_stride   problem b's column indices (and stored values, if s_values is not
 *                    NULL) are col_idx + b * nnz_stride (s_values + b * nnz_stride); nnz_stride is at least
 *                    every problem's entry count (row_ptr_b[M]); with a shared pattern pass nnz_stride = that
 *                    count for the size queries and the family choice -- then s_values is shared too
 *                    (stride 0 is taken when row_ptr_stride is 0)
 *   A, lda, stride_a (and B, D, O likewise)   problem b's operand is A + b * stride_a, row-major with
 *                    leading dimension lda; an input's stride may be 0 (operand shared by all problems);
 *                    outputs must not overlap: stride_o >= (M - 1) * ldo + N
 * Workspace: b2sp_workspace_bytes_batched(...) bytes.  algo as for b2sp_fusedmm; B2SP_ALGO_ROW and
 * B2SP_ALGO_ROW_NAT both take the rows in natural order; B2SP_ALGO_TILE_PREPARED needs a table built by
 * b2sp_prepare_pattern_batched with the same batch, M, K, nnz_stride, row_ptr, row_ptr_stride and col_idx.
 * B2SP_ALGO_AUTO chooses the family from the density nnz_stride / (M * K).  Outputs wider than 256
 * columns (where a single problem takes two phases, see b2sp_fusedmm) run on the row kernels.
 * Every other convention (device pointers, asynchronous on `stream`, outputs overwritten, patterns that
 * are not strictly sorted handled by the row kernels inside the same call) is b2sp_fusedmm's.
 */
size_t b2sp_workspace_bytes_batched(int batch, int M, int K, int Kd, int N, long long nnz_stride);
b2sp_status b2sp_prepare_pattern_batched(int batch, int M, int K, long long nnz_stride, const int *row_ptr,
                                         long long row_ptr_stride, const int *col_idx, void *workspace,
                                         size_t workspace_bytes, void *stream);
b2sp_status b2sp_fusedmm_batched(int batch, int M, int K, int Kd, int N, long long nnz_stride,
                                 const int *row_ptr, long long row_ptr_stride, const int *col_idx,
                                 const float *s_values, const float *A, long long lda, long long stride_a,
                                 const float *B, long long ldb, long long stride_b, const float *D, long long ldd,
                                 long long stride_d, float *O, long long ldo, long long stride_o, void *workspace,
                                 size_t workspace_bytes, int algo, void *stream);
/* The same with bfloat16 A, B, D (see b2sp_fusedmm_bf16): e.g. sparse attention on bfloat16 Q, K, V. */
b2sp_status b2sp_fusedmm_batched_bf16(int batch, int M, int K, int Kd, int N, long long nnz_stride,
                                      const int *row_ptr, long long row_ptr_stride, const int *col_idx,
                                      const float *s_values, const void *A, long long lda, long long stride_a,
                                      const void *B, long long ldb, long long stride_b, const void *D, long long ldd,
                                      long long stride_d, float *O, long long ldo, long long stride_o, void *workspace,
                                      size_t workspace_bytes, int algo, void *stream);

/*
 * Host-buffer forms of the three ops: every data pointer is a HOST pointer (pinned memory
 * makes the copies asynchronous and faster, pageable memory also works).  Each call copies
 * its inputs to the device, runs the device entry point above with algo = B2SP_ALGO_AUTO,
 * copies the result back and synchronises `stream` before returning.  Device memory comes
 * from a stream-ordered memory pool that the library creates for itself on each device at first
 * use (the process's default pool and its settings are not touched) and is returned to that pool
 * before the call ends; the pool keeps freed blocks for the next call.  Dense operands are
 * contiguous (ld = number of columns).  The workspace's device status word is read back with the
 * result: B2SP_ERR_TIMEOUT if a bounded wait inside a kernel gave up (outputs undefined).
 */
b2sp_status b2sp_spmm_host(int M, int K, int N, long long nnz,
                           const int *row_ptr, const int *col_idx, const float *values,
                           const float *D, float *O, void *stream);
b2sp_status b2sp_sddmm_host(int M, int K, int Kd, long long nnz,
                            const int *row_ptr, const int *col_idx, const float *s_values,
                            const float *A, const float *B, float *out_values, void *stream);
b2sp_status b2sp_fusedmm_host(int M, int K, int Kd, int N, long long nnz,
                              const int *row_ptr, const int *col_idx, const float *s_values,
                              const float *A, const float *B, const float *D, float *O,
                              void *stream);

/*
 * SPMM without any allocation, for callers that cannot obtain device memory of their own.
 * (The paper has no counterpart; this is a deployment convenience, not part of its method.)
 *
 * Who needs it: code that runs where cudaMalloc is not an option -- a plug-in inside a serving
 * process that gave all device memory to its own arena at start-up, or a latency-critical loop
 * that must not trigger the device-wide synchronisation an allocation can cause.  Such a caller
 * owns inputs and outputs but has no workspace to offer, so this entry point keeps the row-binning
 * workspace in a fixed array inside the library's device image instead.
 *
 * Same result and same argument meaning as b2sp_spmm with B2SP_ALGO_ROW (all data pointers are
 * device pointers; O is fully overwritten), minus the workspace and algo arguments.
 *
 * Limits and rules:
 *   - M <= B2SP_STATIC_SCRATCH_MAX_ROWS, otherwise B2SP_ERR_TOO_LARGE and nothing is enqueued.
 *     K, N and nnz are unrestricted.
 *   - The array (512 bytes + 4 bytes per row of the limit, about 257 KiB) is part of the library's
 *     device image: every GPU on which the image gets loaded holds it until the process exits.
 *   - The first call on each device looks up the array's device address.  With CUDA's lazy module
 *     loading that look-up is also what loads the library's device image on that GPU, and the
 *     driver reserves room for the array (and the code) at that moment; it may synchronise the
 *     device.  So make the first call at start-up: with the device current, BEFORE the host
 *     process's arena takes the remaining device memory, outside any latency-critical loop and
 *     before starting any stream capture.  Later calls on that device do no such work.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left.  The
 *     part that must start from zero is cleared at the start of each call, so back-to-back calls on
 *     one stream are fine; two calls that can overlap on the GPU (different streams, or different
 *     host threads with different streams) race on it and give wrong results.  Use b2sp_spmm with
 *     separate workspaces for concurrent work.
 *   - The entry point itself calls no cudaMalloc / cudaFree / pool allocator and launches only a
 *     small memset and kernels on `stream`; it does not synchronise.
 */
#define B2SP_STATIC_SCRATCH_MAX_ROWS 65536
b2sp_status b2sp_spmm_static_scratch(int M, int K, int N, long long nnz,
                                     const int *row_ptr, const int *col_idx, const float *values,
                                     const float *D, long long ldd, float *O, long long ldo,
                                     void *stream);

/*
 * Debug helper: checks on the device that row_ptr[0] = 0, row_ptr is non-decreasing,
 * row_ptr[M] = nnz and 0 <= col_idx[p] < K.  Synchronises `stream`.  `workspace` needs 256
 * bytes.  Returns B2SP_OK or B2SP_ERR_BAD_CSR.
 */
b2sp_status b2sp_validate_csr(int M, int K, long long nnz, const int *row_ptr, const int *col_idx,
                              void *workspace, size_t workspace_bytes, void *stream);

/*
 * Reads back (synchronising `stream`) the status word device code left in `workspace` during
 * the most recent op that used it: B2SP_OK, or B2SP_ERR_TIMEOUT if a bounded wait inside a
 * kernel gave up (the outputs of that call are then undefined).
 */
b2sp_status b2sp_device_status(const void *workspace, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* B2SP_H */
