// C-ABI entry points of libb2sp: argument checks, workspace carving, kernel dispatch.
// See include/b2sp.h (and include/b2sp_debug.h) for the contract of every function.
#include "../../include/b2sp_debug.h"

#include <climits>
#include <cstdlib>
#include <cstdint>
#include <mutex>

#include "row_kernels.cuh"
#include "tile_dispatch.h"

namespace b2sp {

// ---- workspace layout ---------------------------------------------------------------------
// [0, 128)    int count[32]      row-length histogram            (zeroed per call)
// [128, 256)  int cursor[32]     scatter cursors                 (zeroed per call)
// [256, 512)  int status[64]     status[0] = device status word, status[1] = validate flag
// [512, ...)  int row_order[M]   rows, longest bucket first
constexpr size_t kHeaderBytes = 512;

inline size_t align256(size_t x) { return (x + 255) & ~size_t(255); }
inline size_t row_workspace_bytes(int M) { return align256(kHeaderBytes + sizeof(int) * (size_t)M); }

struct Workspace {
    int *count, *cursor, *status, *row_order;
};

inline Workspace carve(void *ws)
{
    char *b = static_cast<char *>(ws);
    Workspace w;
    w.count = reinterpret_cast<int *>(b);
    w.cursor = reinterpret_cast<int *>(b + 128);
    w.status = reinterpret_cast<int *>(b + 256);
    w.row_order = reinterpret_cast<int *>(b + kHeaderBytes);
    return w;
}

thread_local int g_last_algo[3] = {-1, -1, -1};
thread_local int g_last_launches[3] = {0, 0, 0};

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
// alignment a dense operand needs for the four-element loads of the vector kernels (16 bytes of fp32, 8 of bf16)
template <typename DT> inline bool aligned_vec(const DT *p) { return (reinterpret_cast<uintptr_t>(p) & (4 * sizeof(DT) - 1)) == 0; }
template <typename DT> constexpr int dense_dtype() { return sizeof(DT) == 2 ? kDenseBf16 : kDenseF32; }

inline b2sp_status check_launch()
{
    return cudaGetLastError() == cudaSuccess ? B2SP_OK : B2SP_ERR_CUDA;
}

b2sp_status check_workspace(void *ws, size_t have, size_t need)
{
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255) != 0 || have < need) return B2SP_ERR_WORKSPACE;
    return B2SP_OK;
}

// Enqueue the binning pass; returns the row order pointer (NULL for natural order).
b2sp_status bin_rows(int M, const int *row_ptr, const Workspace &w, cudaStream_t st, int *launches)
{
    if (cudaMemsetAsync(w.count, 0, 512, st) != cudaSuccess) return B2SP_ERR_CUDA;
    int blocks = (M + 255) / 256;
    bin_count_kernel<<<blocks, 256, 0, st>>>(M, row_ptr, w.count);
    {   // a programmatic dependent of the counting kernel (it waits for the counts where it needs them)
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)blocks);
        cfg.blockDim = dim3(256);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaLaunchKernelEx(&cfg, bin_scatter_kernel, M, row_ptr, (const int *)w.count, w.cursor, w.row_order);
    }
    *launches += 2;
    return check_launch();
}

// Launches `kern`; a gated launch (the row family as the dense-tile family's device-side fallback) is marked as a
// programmatic dependent of the tile kernel before it: the tile kernel lets its dependents go as soon
// as it has read the gate's flags, which are final before it starts, so the fallback (which almost always
// finds its gate closed and exits) runs beside the tile kernel instead of after it.  A launch behind the binning
// pass (`order` given) is a programmatic dependent of it too: the kernel waits for the row order at its top.
template <class... KArgs, class... Args>
inline void launch_row(void (*kern)(KArgs...), dim3 grid, size_t smem, cudaStream_t st, bool dependent, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kRowThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = dependent ? attr : nullptr;
    cfg.numAttrs = dependent ? 1 : 0;
    cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

// A gated launch (the row family as the dense-tile family's fallback) almost always finds its gate
// closed: it gets a small grid whose blocks walk the rows, so that the usual case costs little.
inline unsigned gated_blocks(unsigned rows, int *gate, unsigned nbatch = 1)
{
    unsigned cap = 148u * 4u / (nbatch ? nbatch : 1);   // (every CTA of a gated grid counts itself at the gate: keep them few)
    if (cap < 16u) cap = 16u;
    return gate && rows > cap ? cap : rows;
}

template <int U, int SPLIT, typename DT>
void launch_spmm(dim3 grid, cudaStream_t st, int N, const int *row_ptr, const int *col_idx,
                 const float *values, const DT *D, int64_t ldd, float *O, int64_t ldo,
                 const int *order, int *gate, int *clear)
{
    const int nrows = (int)grid.x;
    grid.x = gated_blocks(grid.x, gate);
    launch_row(spmm_row_kernel<U, SPLIT, DT>, grid, 0, st, gate != nullptr || order != nullptr, N, row_ptr, col_idx, values, D, ldd, O, ldo, order,
               gate, nrows, clear);
}

// Column geometry for a width N on the float4 path: U float4 per lane, SPLIT sub-warps.
struct Geom { int U, SPLIT, slab; };
inline Geom pick_geom(int N)
{
    if (N <= 32) return {1, 4, 32};
    if (N <= 64) return {1, 2, 64};
    if (N <= 128) return {1, 1, 128};
    if (N <= 256) return {2, 1, 256};
    return {4, 1, 512};
}

inline int pick_ku(int Kd) { return Kd <= 64 ? 2 : Kd <= 128 ? 4 : Kd <= 256 ? 8 : 0; }

template <int KU, typename DT>
void launch_sddmm(dim3 grid, cudaStream_t st, int Kd, const int *row_ptr, const int *col_idx,
                  const float *sv, const DT *A, int64_t lda, const DT *B, int64_t ldb,
                  float *out, const int *order, int *gate, int *clear)
{
    size_t smem = KU == 0 ? sizeof(float) * (size_t)((Kd + 3) & ~3) : 0;
    const int nrows = (int)grid.x;
    grid.x = gated_blocks(grid.x, gate);
    launch_row(sddmm_row_kernel<KU, DT>, grid, smem, st, gate != nullptr || order != nullptr, Kd, row_ptr, col_idx, sv, A, lda, B, ldb, out, order,
               gate, nrows, clear);
}

template <int KU, int U, int SPLIT, typename DT>
b2sp_status launch_fused(dim3 grid, cudaStream_t st, int Kd, int N, const int *row_ptr,
                         const int *col_idx, const float *sv, const DT *A, int64_t lda,
                         const DT *B, int64_t ldb, const DT *D, int64_t ldd, float *O,
                         int64_t ldo, const int *order, int *gate, int *clear, const RowBatch &rb)
{
    size_t smem = sizeof(float4) * kRowWarps * U * (32 / SPLIT) +
                  (KU == 0 ? sizeof(float) * (size_t)((Kd + 3) & ~3) : 0);
    const bool batched = grid.z > 1;
    auto kern_b = fusedmm_row_kernel<KU, U, SPLIT, true, DT>;
    auto kern_1 = fusedmm_row_kernel<KU, U, SPLIT, false, DT>;
    if (smem > 48 * 1024) {
        if (smem > 200 * 1024) return B2SP_ERR_UNSUPPORTED;
        if (cudaFuncSetAttribute(batched ? reinterpret_cast<const void *>(kern_b) : reinterpret_cast<const void *>(kern_1),
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return B2SP_ERR_CUDA;
    }
    const int nrows = (int)grid.x;
    grid.x = gated_blocks(grid.x, gate, grid.z);
    if (batched)
        launch_row(kern_b, grid, smem, st, gate != nullptr || order != nullptr, Kd, N, row_ptr, col_idx, sv, A, lda, B, ldb, D, ldd, O, ldo,
                   order, gate, nrows, clear, rb);
    else
        launch_row(kern_1, grid, smem, st, gate != nullptr || order != nullptr, Kd, N, row_ptr, col_idx, sv, A, lda, B, ldb, D, ldd, O, ldo,
                   order, gate, nrows, clear, NoBatch{});
    return B2SP_OK;
}

template <int KU, typename DT>
b2sp_status dispatch_fused_geom(const Geom &g, dim3 grid, cudaStream_t st, int Kd, int N,
                                const int *row_ptr, const int *col_idx, const float *sv,
                                const DT *A, int64_t lda, const DT *B, int64_t ldb,
                                const DT *D, int64_t ldd, float *O, int64_t ldo,
                                const int *order, int *gate, int *clear, const RowBatch &rb)
{
#define B2SP_F(U_, S_) \
    return launch_fused<KU, U_, S_, DT>(grid, st, Kd, N, row_ptr, col_idx, sv, A, lda, B, ldb, D, ldd, O, ldo, order, gate, clear, rb)
    if (g.SPLIT == 4) B2SP_F(1, 4);
    if (g.SPLIT == 2) B2SP_F(1, 2);
    if (g.U == 1) B2SP_F(1, 1);
    if (g.U == 2) B2SP_F(2, 1);
    B2SP_F(4, 1);
#undef B2SP_F
}

b2sp_status zero_rows(float *O, int64_t ldo, int M, int N, cudaStream_t st)
{
    if (M == 0 || N == 0) return B2SP_OK;
    return cudaMemset2DAsync(O, sizeof(float) * (size_t)ldo, 0, sizeof(float) * (size_t)N, (size_t)M,
                             st) == cudaSuccess
               ? B2SP_OK
               : B2SP_ERR_CUDA;
}

bool bad_csr_args(int M, int K, long long nnz, const int *row_ptr, const int *col_idx)
{
    if (M < 0 || K < 0 || nnz < 0 || nnz > (long long)INT_MAX) return true;
    if (M > 0 && !row_ptr) return true;
    if (nnz > 0 && (!col_idx || K == 0 || M == 0)) return true;
    return false;
}

}  // namespace b2sp

using namespace b2sp;

extern "C" int b2sp_version(void) { return 100; }

extern "C" const char *b2sp_status_string(b2sp_status s)
{
    switch (s) {
    case B2SP_OK: return "ok";
    case B2SP_ERR_INVALID_ARG: return "invalid argument";
    case B2SP_ERR_UNSUPPORTED: return "unsupported for these arguments";
    case B2SP_ERR_BAD_CSR: return "malformed CSR";
    case B2SP_ERR_CUDA: return "CUDA error";
    case B2SP_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case B2SP_ERR_TIMEOUT: return "device-side wait timed out";
    case B2SP_ERR_TOO_LARGE: return "problem exceeds the library's built-in scratch array";
    }
    return "unknown status";
}

// The FusedMM tile kernel owns one 128-column tile of O and recomputes S (.) A B^T for each of them
// (tensor memory holds O, P, P' and A for one tile only).  Past two tiles that costs more than
// writing the sampled values once: measured at N = 512 on the 8192^2 / 30% workload, 717 us fused
// against 134 + 430 us for SDDMM into a scratch C and SPMM on C.  So wide outputs take the two
// phases inside one call (same window table, same fallback), and C lives in the workspace.
// With two tiles (128 < N <= 256) the second GEMM1 costs more than C's round trip when GEMM1 is long and the
// problem large: measured at N = 256, Kd = 128, two phases against fused: 8192^2 315 against 342 us (10% density
// 298 against 337), 4096 x 8192 175 against 188, 16384 x 2048 187 against 191, 4096^2 115 against 114; but
// 8192 x 4096 at Kd = 64 172 against 159 and 2048^2 52 against 40.
static bool fusedmm_two_phase(int M, int K, int Kd, int N)
{
    return N > 256 || (N > 128 && Kd > 64 && (double)M * (double)K >= 3.0e7);
}

// Workspace of the dense-tile family for an op (0: these sizes are outside the family).
static size_t tile_workspace_bytes(int op, int M, int K, int Kd, int N, long long nnz, size_t row_bytes)
{
    FusedPlan p = op == B2SP_OP_SPMM    ? plan_fused_tile(M, K, 0, N, nnz, row_bytes, true)
                  : op == B2SP_OP_SDDMM ? plan_fused_tile(M, K, Kd, 0, nnz, row_bytes, false)
                                        : plan_fused_tile(M, K, Kd, N, nnz, row_bytes, true);
    if (!p.feasible) return 0;
    if (op == B2SP_OP_FUSEDMM && fusedmm_two_phase(M, K, Kd, N)) {
        TwoPhasePlan t = plan_two_phase(M, K, Kd, N, nnz, row_bytes);
        if (t.feasible && t.bytes > p.bytes) return t.bytes;
    }
    return p.bytes;
}

static int tile_width(int op, int Kd, int N) { return op == B2SP_OP_SPMM ? N : op == B2SP_OP_SDDMM ? Kd : (Kd < N ? Kd : N); }

extern "C" size_t b2sp_workspace_bytes_algo(int op, int algo, int M, int K, int Kd, int N, long long nnz)
{
    if (op < 0 || op > 2 || M < 0 || K < 0 || Kd < 0 || N < 0 || nnz < 0) return 0;
    if (algo < B2SP_ALGO_AUTO || algo > B2SP_ALGO_TILE_PREPARED) return 0;
    const size_t rows = row_workspace_bytes(M);
    if (algo == B2SP_ALGO_ROW || algo == B2SP_ALGO_ROW_NAT) return rows;
    const size_t tile = tile_workspace_bytes(op, M, K, Kd, N, nnz, rows);
    if (algo == B2SP_ALGO_TILE || algo == B2SP_ALGO_TILE_PREPARED) return tile;
    return tile > rows && tile_profitable(op, M, K, tile_width(op, Kd, N), nnz) ? tile : rows;
}

extern "C" size_t b2sp_workspace_bytes(int op, int M, int K, int Kd, int N, long long nnz)
{
    if (op < 0 || op > 2 || M < 0 || K < 0 || Kd < 0 || N < 0 || nnz < 0) return 0;
    const size_t rows = row_workspace_bytes(M);
    const size_t tile = tile_workspace_bytes(op, M, K, Kd, N, nnz, rows);
    return tile > rows ? tile : rows;
}

extern "C" int b2sp_last_algo(int op) { return op >= 0 && op < 3 ? g_last_algo[op] : -1; }
extern "C" int b2sp_last_launches(int op) { return op >= 0 && op < 3 ? g_last_launches[op] : 0; }

// The row family under AUTO: the binning pass (two small launches, ~10 us) orders the rows longest
// first, which only pays when the CTAs of the row kernel need several waves on the GPU.
static int auto_row_algo(int M) { return M <= 4096 ? B2SP_ALGO_ROW_NAT : B2SP_ALGO_ROW; }

// Enqueues the row-family SPMM.  `gate` != NULL makes it a device-side fallback.
template <typename DT>
static b2sp_status spmm_rows(int M, int N, const int *row_ptr, const int *col_idx, const float *values,
                             const DT *D, long long ldd, float *O, long long ldo, const int *order,
                             int *gate, int *clear, cudaStream_t st)
{
    bool vec = N % 4 == 0 && ldd % 4 == 0 && ldo % 4 == 0 && aligned_vec(D) && aligned16(O);
    if (vec) {
        Geom g = pick_geom(N);
        dim3 grid((unsigned)M, (unsigned)((N + g.slab - 1) / g.slab));
        if (g.SPLIT == 4) launch_spmm<1, 4, DT>(grid, st, N, row_ptr, col_idx, values, D, ldd, O, ldo, order, gate, clear);
        else if (g.SPLIT == 2) launch_spmm<1, 2, DT>(grid, st, N, row_ptr, col_idx, values, D, ldd, O, ldo, order, gate, clear);
        else if (g.U == 1) launch_spmm<1, 1, DT>(grid, st, N, row_ptr, col_idx, values, D, ldd, O, ldo, order, gate, clear);
        else if (g.U == 2) launch_spmm<2, 1, DT>(grid, st, N, row_ptr, col_idx, values, D, ldd, O, ldo, order, gate, clear);
        else launch_spmm<4, 1, DT>(grid, st, N, row_ptr, col_idx, values, D, ldd, O, ldo, order, gate, clear);
    } else {
        dim3 grid(gated_blocks((unsigned)M, gate), (unsigned)((N + 127) / 128));
        launch_row(spmm_row_scalar_kernel<DT>, grid, 0, st, gate != nullptr || order != nullptr, N, row_ptr, col_idx, values, D, ldd, O, ldo, order,
                   gate, M, clear);
    }
    return check_launch();
}

template <typename DT>
static b2sp_status spmm_impl(int M, int K, int N, long long nnz, const int *row_ptr, const int *col_idx,
                             const float *values, const DT *D, long long ldd, float *O, long long ldo,
                             void *workspace, size_t workspace_bytes, int algo, void *stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (bad_csr_args(M, K, nnz, row_ptr, col_idx) || N < 0) return B2SP_ERR_INVALID_ARG;
    if (algo < B2SP_ALGO_AUTO || algo > B2SP_ALGO_TILE_PREPARED) return B2SP_ERR_INVALID_ARG;
    const bool prepared = algo == B2SP_ALGO_TILE_PREPARED;
    if (prepared) algo = B2SP_ALGO_TILE;
    if (M > 0 && N > 0 && (!O || ldo < N)) return B2SP_ERR_INVALID_ARG;
    if (nnz > 0 && N > 0 && (!values || !D || ldd < N)) return B2SP_ERR_INVALID_ARG;
    const size_t row_bytes = row_workspace_bytes(M);
    b2sp_status rc = check_workspace(workspace, workspace_bytes, row_bytes);
    if (rc != B2SP_OK) return rc;
    FusedPlan plan;   // SPMM runs through the FusedMM tile pipeline with P' = the stored values (Kd = 0)
    if (algo == B2SP_ALGO_TILE || (algo == B2SP_ALGO_AUTO && tile_profitable(B2SP_OP_SPMM, M, K, N, nnz)))
        plan = plan_fused_tile(M, K, 0, N, nnz, row_bytes, true);
    int use = algo == B2SP_ALGO_AUTO ? auto_row_algo(M) : algo;
    if (plan.feasible && workspace_bytes >= plan.bytes) use = B2SP_ALGO_TILE;
    else if (algo == B2SP_ALGO_TILE) return plan.feasible ? B2SP_ERR_WORKSPACE : B2SP_ERR_UNSUPPORTED;
    g_last_algo[B2SP_OP_SPMM] = use;
    int launches = 0;
    g_last_launches[B2SP_OP_SPMM] = 0;
    if (M == 0 || N == 0) return B2SP_OK;
    if (nnz == 0) return zero_rows(O, ldo, M, N, st);

    Workspace w = carve(workspace);
    if (use == B2SP_ALGO_TILE) {
        rc = fused_tile(plan, prepared, 2, M, K, 0, N, nnz, row_ptr, col_idx, values, nullptr, 0, nullptr, 0, D, ldd,
                        O, ldo, workspace, st, &launches, false, BatchDesc(), dense_dtype<DT>());
        if (rc != B2SP_OK) return rc;
        // device-side fallback: runs only if the pre-pass found rows that are not strictly sorted
        int *gate = reinterpret_cast<int *>(static_cast<char *>(workspace) + kWsTileFlagsOffset);
        rc = spmm_rows(M, N, row_ptr, col_idx, values, D, ldd, O, ldo, nullptr, gate, nullptr, st);
        g_last_launches[B2SP_OP_SPMM] = launches + 1;
        return rc;
    }
    const int *order = nullptr;
    int *clear = nullptr;
    if (use == B2SP_ALGO_ROW) {
        rc = bin_rows(M, row_ptr, w, st, &launches);
        if (rc != B2SP_OK) return rc;
        order = w.row_order;
    } else {   // no binning pass: the row kernel itself resets the status word
        clear = reinterpret_cast<int *>(static_cast<char *>(workspace) + kWsStatusOffset);
    }
    rc = spmm_rows(M, N, row_ptr, col_idx, values, D, ldd, O, ldo, order, nullptr, clear, st);
    g_last_launches[B2SP_OP_SPMM] = launches + 1;
    return rc;
}

// Enqueues the row-family SDDMM.  `gate` != NULL makes it a device-side fallback.
template <typename DT>
static b2sp_status sddmm_rows(int M, int Kd, const int *row_ptr, const int *col_idx, const float *s_values,
                              const DT *A, long long lda, const DT *B, long long ldb,
                              float *out_values, const int *order, int *gate, int *clear, cudaStream_t st)
{
    dim3 grid((unsigned)M);
    bool vec = Kd % 4 == 0 && lda % 4 == 0 && ldb % 4 == 0 && aligned_vec(A) && aligned_vec(B) &&
               Kd <= 40960;
    if (vec) {
        switch (pick_ku(Kd)) {
        case 2: launch_sddmm<2, DT>(grid, st, Kd, row_ptr, col_idx, s_values, A, lda, B, ldb, out_values, order, gate, clear); break;
        case 4: launch_sddmm<4, DT>(grid, st, Kd, row_ptr, col_idx, s_values, A, lda, B, ldb, out_values, order, gate, clear); break;
        case 8: launch_sddmm<8, DT>(grid, st, Kd, row_ptr, col_idx, s_values, A, lda, B, ldb, out_values, order, gate, clear); break;
        default: {
            size_t smem = sizeof(float) * (size_t)Kd;
            if (smem > 48 * 1024 &&
                cudaFuncSetAttribute(sddmm_row_kernel<0, DT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)smem) != cudaSuccess)
                return B2SP_ERR_CUDA;
            launch_sddmm<0, DT>(grid, st, Kd, row_ptr, col_idx, s_values, A, lda, B, ldb, out_values, order, gate, clear);
        }
        }
    } else {
        grid.x = gated_blocks(grid.x, gate);
        launch_row(sddmm_row_scalar_kernel<DT>, grid, 0, st, gate != nullptr || order != nullptr, Kd, row_ptr, col_idx, s_values, A, lda, B, ldb,
                   out_values, order, gate, M, clear);
    }
    return check_launch();
}

template <typename DT>
static b2sp_status sddmm_impl(int M, int K, int Kd, long long nnz, const int *row_ptr, const int *col_idx,
                              const float *s_values, const DT *A, long long lda, const DT *B,
                              long long ldb, float *out_values, void *workspace, size_t workspace_bytes,
                              int algo, void *stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (bad_csr_args(M, K, nnz, row_ptr, col_idx) || Kd < 0) return B2SP_ERR_INVALID_ARG;
    if (algo < B2SP_ALGO_AUTO || algo > B2SP_ALGO_TILE_PREPARED) return B2SP_ERR_INVALID_ARG;
    const bool prepared = algo == B2SP_ALGO_TILE_PREPARED;
    if (prepared) algo = B2SP_ALGO_TILE;
    if (nnz > 0 && !out_values) return B2SP_ERR_INVALID_ARG;
    if (nnz > 0 && Kd > 0 && (!A || !B || lda < Kd || ldb < Kd)) return B2SP_ERR_INVALID_ARG;
    const size_t row_bytes = row_workspace_bytes(M);
    b2sp_status rc = check_workspace(workspace, workspace_bytes, row_bytes);
    if (rc != B2SP_OK) return rc;
    FusedPlan plan;
    if (algo == B2SP_ALGO_TILE || (algo == B2SP_ALGO_AUTO && tile_profitable(B2SP_OP_SDDMM, M, K, Kd, nnz)))
        plan = plan_fused_tile(M, K, Kd, 0, nnz, row_bytes, false);
    int use = algo == B2SP_ALGO_AUTO ? auto_row_algo(M) : algo;
    if (plan.feasible && workspace_bytes >= plan.bytes) use = B2SP_ALGO_TILE;
    else if (algo == B2SP_ALGO_TILE) return plan.feasible ? B2SP_ERR_WORKSPACE : B2SP_ERR_UNSUPPORTED;
    g_last_algo[B2SP_OP_SDDMM] = use;
    int launches = 0;
    g_last_launches[B2SP_OP_SDDMM] = 0;
    if (M == 0 || nnz == 0) return B2SP_OK;
    if (Kd == 0)
        return cudaMemsetAsync(out_values, 0, sizeof(float) * (size_t)nnz, st) == cudaSuccess
                   ? B2SP_OK
                   : B2SP_ERR_CUDA;

    Workspace w = carve(workspace);
    if (use == B2SP_ALGO_TILE) {
        rc = fused_tile(plan, prepared, 0, M, K, Kd, 0, nnz, row_ptr, col_idx, s_values, A, lda, B, ldb, nullptr, 0,
                        out_values, 0, workspace, st, &launches, false, BatchDesc(), dense_dtype<DT>());
        if (rc != B2SP_OK) return rc;
        int *gate = reinterpret_cast<int *>(static_cast<char *>(workspace) + kWsTileFlagsOffset);
        rc = sddmm_rows(M, Kd, row_ptr, col_idx, s_values, A, lda, B, ldb, out_values, nullptr, gate, nullptr, st);
        g_last_launches[B2SP_OP_SDDMM] = launches + 1;
        return rc;
    }
    const int *order = nullptr;
    int *clear = nullptr;
    if (use == B2SP_ALGO_ROW) {
        rc = bin_rows(M, row_ptr, w, st, &launches);
        if (rc != B2SP_OK) return rc;
        order = w.row_order;
    } else {   // no binning pass: the row kernel itself resets the status word
        clear = reinterpret_cast<int *>(static_cast<char *>(workspace) + kWsStatusOffset);
    }
    rc = sddmm_rows(M, Kd, row_ptr, col_idx, s_values, A, lda, B, ldb, out_values, order, nullptr, clear, st);
    g_last_launches[B2SP_OP_SDDMM] = launches + 1;
    return rc;
}

// Enqueues the row-family FusedMM.  `gate` != NULL makes it a device-side fallback.
template <typename DT>
static b2sp_status fused_rows(int M, int Kd, int N, const int *row_ptr, const int *col_idx,
                              const float *s_values, const DT *A, long long lda, const DT *B,
                              long long ldb, const DT *D, long long ldd, float *O, long long ldo,
                              const int *order, int *gate, int *clear, cudaStream_t st,
                              int nbatch = 1, const RowBatch &rb = RowBatch{0, 0, 0, 0, 0, 0})
{
    b2sp_status rc = B2SP_OK;
    bool vec = N % 4 == 0 && ldd % 4 == 0 && ldo % 4 == 0 && aligned_vec(D) && aligned16(O) &&
               Kd % 4 == 0 && lda % 4 == 0 && ldb % 4 == 0 && aligned_vec(A) && aligned_vec(B) &&
               Kd <= 40960 && ((rb.A | rb.B | rb.D | rb.O) & 3) == 0;
    if (vec) {
        Geom g = pick_geom(N);
        dim3 grid((unsigned)M, (unsigned)((N + g.slab - 1) / g.slab), (unsigned)nbatch);
        switch (pick_ku(Kd)) {
        case 2: rc = dispatch_fused_geom<2, DT>(g, grid, st, Kd, N, row_ptr, col_idx, s_values, A, lda, B, ldb, D, ldd, O, ldo, order, gate, clear, rb); break;
        case 4: rc = dispatch_fused_geom<4, DT>(g, grid, st, Kd, N, row_ptr, col_idx, s_values, A, lda, B, ldb, D, ldd, O, ldo, order, gate, clear, rb); break;
        case 8: rc = dispatch_fused_geom<8, DT>(g, grid, st, Kd, N, row_ptr, col_idx, s_values, A, lda, B, ldb, D, ldd, O, ldo, order, gate, clear, rb); break;
        default: rc = dispatch_fused_geom<0, DT>(g, grid, st, Kd, N, row_ptr, col_idx, s_values, A, lda, B, ldb, D, ldd, O, ldo, order, gate, clear, rb); break;
        }
        if (rc != B2SP_OK) return rc;
    } else {
        dim3 grid(gated_blocks((unsigned)M, gate, (unsigned)nbatch), (unsigned)((N + 127) / 128), (unsigned)nbatch);
        launch_row(fusedmm_row_scalar_kernel<DT>, grid, 0, st, gate != nullptr || order != nullptr, Kd, N, row_ptr, col_idx, s_values, A, lda, B, ldb,
                   D, ldd, O, ldo, order, gate, M, clear, rb);
    }
    return check_launch();
}

template <typename DT>
static b2sp_status fusedmm_impl(int M, int K, int Kd, int N, long long nnz, const int *row_ptr,
                                const int *col_idx, const float *s_values, const DT *A, long long lda,
                                const DT *B, long long ldb, const DT *D, long long ldd, float *O,
                                long long ldo, void *workspace, size_t workspace_bytes, int algo,
                                void *stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (bad_csr_args(M, K, nnz, row_ptr, col_idx) || Kd < 0 || N < 0) return B2SP_ERR_INVALID_ARG;
    if (algo < B2SP_ALGO_AUTO || algo > B2SP_ALGO_TILE_PREPARED) return B2SP_ERR_INVALID_ARG;
    const bool prepared = algo == B2SP_ALGO_TILE_PREPARED;
    if (prepared) algo = B2SP_ALGO_TILE;
    if (M > 0 && N > 0 && (!O || ldo < N)) return B2SP_ERR_INVALID_ARG;
    if (nnz > 0 && N > 0 && (!D || ldd < N)) return B2SP_ERR_INVALID_ARG;
    if (nnz > 0 && N > 0 && Kd > 0 && (!A || !B || lda < Kd || ldb < Kd)) return B2SP_ERR_INVALID_ARG;
    const size_t row_bytes = row_workspace_bytes(M);
    b2sp_status rc = check_workspace(workspace, workspace_bytes, row_bytes);
    if (rc != B2SP_OK) return rc;
    FusedPlan plan;
    if (algo == B2SP_ALGO_TILE || (algo == B2SP_ALGO_AUTO && tile_profitable(B2SP_OP_FUSEDMM, M, K, Kd < N ? Kd : N, nnz)))
        plan = plan_fused_tile(M, K, Kd, N, nnz, row_bytes, true);
    int use = algo == B2SP_ALGO_AUTO ? auto_row_algo(M) : algo;
    if (plan.feasible && workspace_bytes >= plan.bytes) use = B2SP_ALGO_TILE;
    else if (algo == B2SP_ALGO_TILE) return plan.feasible ? B2SP_ERR_WORKSPACE : B2SP_ERR_UNSUPPORTED;
    g_last_algo[B2SP_OP_FUSEDMM] = use;
    int launches = 0;
    g_last_launches[B2SP_OP_FUSEDMM] = 0;
    if (M == 0 || N == 0) return B2SP_OK;
    if (nnz == 0 || Kd == 0) return zero_rows(O, ldo, M, N, st);  // empty dot products are 0

    Workspace w = carve(workspace);
    if (use == B2SP_ALGO_TILE) {
        TwoPhasePlan two;
        if (fusedmm_two_phase(M, K, Kd, N)) two = plan_two_phase(M, K, Kd, N, nnz, row_bytes);
        if (two.feasible && workspace_bytes >= two.bytes) {
            float *C = reinterpret_cast<float *>(static_cast<char *>(workspace) + two.off_c);
            rc = fused_tile(two.sddmm, prepared, 0, M, K, Kd, 0, nnz, row_ptr, col_idx, s_values, A, lda, B, ldb, nullptr, 0,
                            C, 0, workspace, st, &launches, false, BatchDesc(), dense_dtype<DT>());
            if (rc != B2SP_OK) return rc;
            rc = fused_tile(two.spmm, true, 2, M, K, 0, N, nnz, row_ptr, col_idx, C, nullptr, 0, nullptr, 0, D, ldd, O, ldo,
                            workspace, st, &launches, /*keep_status=*/true, BatchDesc(), dense_dtype<DT>());
        } else {
            rc = fused_tile(plan, prepared, 1, M, K, Kd, N, nnz, row_ptr, col_idx, s_values, A, lda, B, ldb, D, ldd, O, ldo,
                            workspace, st, &launches, false, BatchDesc(), dense_dtype<DT>());
        }
        if (rc != B2SP_OK) return rc;
        int *gate = reinterpret_cast<int *>(static_cast<char *>(workspace) + kWsTileFlagsOffset);
        rc = fused_rows(M, Kd, N, row_ptr, col_idx, s_values, A, lda, B, ldb, D, ldd, O, ldo, nullptr, gate, nullptr, st);
        g_last_launches[B2SP_OP_FUSEDMM] = launches + 1;
        return rc;
    }
    const int *order = nullptr;
    int *clear = nullptr;
    if (use == B2SP_ALGO_ROW) {
        rc = bin_rows(M, row_ptr, w, st, &launches);
        if (rc != B2SP_OK) return rc;
        order = w.row_order;
    } else {   // no binning pass: the row kernel itself resets the status word
        clear = reinterpret_cast<int *>(static_cast<char *>(workspace) + kWsStatusOffset);
    }
    rc = fused_rows(M, Kd, N, row_ptr, col_idx, s_values, A, lda, B, ldb, D, ldd, O, ldo, order, nullptr, clear, st);
    g_last_launches[B2SP_OP_FUSEDMM] = launches + 1;
    return rc;
}

// ---- the entry points: fp32 and bfloat16 dense operands -------------------------------------------------
extern "C" b2sp_status b2sp_spmm(int M, int K, int N, long long nnz, const int *row_ptr, const int *col_idx,
                                 const float *values, const float *D, long long ldd, float *O, long long ldo,
                                 void *workspace, size_t workspace_bytes, int algo, void *stream)
{
    return spmm_impl<float>(M, K, N, nnz, row_ptr, col_idx, values, D, ldd, O, ldo, workspace, workspace_bytes, algo, stream);
}
extern "C" b2sp_status b2sp_sddmm(int M, int K, int Kd, long long nnz, const int *row_ptr, const int *col_idx,
                                  const float *s_values, const float *A, long long lda, const float *B,
                                  long long ldb, float *out_values, void *workspace, size_t workspace_bytes,
                                  int algo, void *stream)
{
    return sddmm_impl<float>(M, K, Kd, nnz, row_ptr, col_idx, s_values, A, lda, B, ldb, out_values, workspace,
                             workspace_bytes, algo, stream);
}
extern "C" b2sp_status b2sp_fusedmm(int M, int K, int Kd, int N, long long nnz, const int *row_ptr,
                                    const int *col_idx, const float *s_values, const float *A, long long lda,
                                    const float *B, long long ldb, const float *D, long long ldd, float *O,
                                    long long ldo, void *workspace, size_t workspace_bytes, int algo,
                                    void *stream)
{
    return fusedmm_impl<float>(M, K, Kd, N, nnz, row_ptr, col_idx, s_values, A, lda, B, ldb, D, ldd, O, ldo, workspace,
                               workspace_bytes, algo, stream);
}
extern "C" b2sp_status b2sp_spmm_bf16(int M, int K, int N, long long nnz, const int *row_ptr, const int *col_idx,
                                      const float *values, const void *D, long long ldd, float *O, long long ldo,
                                      void *workspace, size_t workspace_bytes, int algo, void *stream)
{
    return spmm_impl<bf16_t>(M, K, N, nnz, row_ptr, col_idx, values, static_cast<const bf16_t *>(D), ldd, O, ldo,
                             workspace, workspace_bytes, algo, stream);
}
extern "C" b2sp_status b2sp_sddmm_bf16(int M, int K, int Kd, long long nnz, const int *row_ptr, const int *col_idx,
                                       const float *s_values, const void *A, long long lda, const void *B,
                                       long long ldb, float *out_values, void *workspace, size_t workspace_bytes,
                                       int algo, void *stream)
{
    return sddmm_impl<bf16_t>(M, K, Kd, nnz, row_ptr, col_idx, s_values, static_cast<const bf16_t *>(A), lda,
                              static_cast<const bf16_t *>(B), ldb, out_values, workspace, workspace_bytes, algo, stream);
}
extern "C" b2sp_status b2sp_fusedmm_bf16(int M, int K, int Kd, int N, long long nnz, const int *row_ptr,
                                         const int *col_idx, const float *s_values, const void *A, long long lda,
                                         const void *B, long long ldb, const void *D, long long ldd, float *O,
                                         long long ldo, void *workspace, size_t workspace_bytes, int algo,
                                         void *stream)
{
    return fusedmm_impl<bf16_t>(M, K, Kd, N, nnz, row_ptr, col_idx, s_values, static_cast<const bf16_t *>(A), lda,
                                static_cast<const bf16_t *>(B), ldb, static_cast<const bf16_t *>(D), ldd, O, ldo,
                                workspace, workspace_bytes, algo, stream);
}

// ---- batched FusedMM --------------------------------------------------------------------------------
namespace {

bool bad_batch_args(int batch, int M, int K, long long nnz_stride, const int *row_ptr, long long row_ptr_stride,
                    const int *col_idx)
{
    if (batch < 1 || M < 0 || K < 0 || nnz_stride < 0 || nnz_stride > (long long)INT_MAX) return true;
    if (M > 0 && !row_ptr) return true;
    if (row_ptr_stride != 0 && row_ptr_stride < (long long)M + 1) return true;
    if (nnz_stride > 0 && (!col_idx || K == 0 || M == 0)) return true;
    return false;
}

FusedPlan plan_batched(int batch, int M, int K, int Kd, int N, long long nnz_stride)
{
    if (N > 256) return FusedPlan();   // wide outputs: not on the dense-tile family in a batch
    return plan_fused_tile(M, K, Kd, N, nnz_stride, row_workspace_bytes(M), true, batch);
}

}  // namespace

extern "C" size_t b2sp_workspace_bytes_batched(int batch, int M, int K, int Kd, int N, long long nnz_stride)
{
    if (batch < 1 || M < 0 || K < 0 || Kd < 0 || N < 0 || nnz_stride < 0) return 0;
    const size_t rows = row_workspace_bytes(M);
    const FusedPlan p = plan_batched(batch, M, K, Kd, N, nnz_stride);
    return p.feasible && p.bytes > rows ? p.bytes : rows;
}

extern "C" b2sp_status b2sp_prepare_pattern_batched(int batch, int M, int K, long long nnz_stride, const int *row_ptr,
                                         long long row_ptr_stride, const int *col_idx, void *workspace,
                                         size_t workspace_bytes, void *stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (bad_batch_args(batch, M, K, nnz_stride, row_ptr, row_ptr_stride, col_idx) || M == 0 || K == 0 || nnz_stride == 0)
        return B2SP_ERR_INVALID_ARG;
    const size_t need = pattern_table_offset(M) + pattern_table_bytes(M, K, batch);
    b2sp_status rc = check_workspace(workspace, workspace_bytes, need);
    if (rc != B2SP_OK) return rc;
    int launches = 0;
    BatchDesc bd;
    bd.count = batch; bd.rp = row_ptr_stride; bd.nz = row_ptr_stride == 0 ? 0 : nnz_stride;   // a shared pattern
    return pattern_pass(false, M, K, nnz_stride, row_ptr, col_idx, workspace, st, &launches, bd);
}

template <typename DT>
static b2sp_status fusedmm_batched_impl(int batch, int M, int K, int Kd, int N, long long nnz_stride,
                                        const int *row_ptr, long long row_ptr_stride, const int *col_idx,
                                        const float *s_values, const DT *A, long long lda, long long stride_a,
                                        const DT *B, long long ldb, long long stride_b, const DT *D, long long ldd,
                                        long long stride_d, float *O, long long ldo, long long stride_o, void *workspace,
                                        size_t workspace_bytes, int algo, void *stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (bad_batch_args(batch, M, K, nnz_stride, row_ptr, row_ptr_stride, col_idx) || Kd < 0 || N < 0)
        return B2SP_ERR_INVALID_ARG;
    if (algo < B2SP_ALGO_AUTO || algo > B2SP_ALGO_TILE_PREPARED) return B2SP_ERR_INVALID_ARG;
    const bool prepared = algo == B2SP_ALGO_TILE_PREPARED;
    if (prepared) algo = B2SP_ALGO_TILE;
    if (stride_a < 0 || stride_b < 0 || stride_d < 0) return B2SP_ERR_INVALID_ARG;
    if (M > 0 && N > 0 && (!O || ldo < N || (batch > 1 && stride_o < (long long)(M - 1) * ldo + N))) return B2SP_ERR_INVALID_ARG;
    if (nnz_stride > 0 && N > 0 && (!D || ldd < N)) return B2SP_ERR_INVALID_ARG;
    if (nnz_stride > 0 && N > 0 && Kd > 0 && (!A || !B || lda < Kd || ldb < Kd)) return B2SP_ERR_INVALID_ARG;
    const size_t row_bytes = row_workspace_bytes(M);
    b2sp_status rc = check_workspace(workspace, workspace_bytes, row_bytes);
    if (rc != B2SP_OK) return rc;
    FusedPlan plan;
    // (the family is chosen from nnz_stride, an upper bound of every problem's entry count)
    if (algo == B2SP_ALGO_TILE ||
        (algo == B2SP_ALGO_AUTO && tile_profitable(B2SP_OP_FUSEDMM, M, K, Kd < N ? Kd : N, nnz_stride)))
        plan = plan_batched(batch, M, K, Kd, N, nnz_stride);
    int use = B2SP_ALGO_ROW_NAT;   // the row family takes the problems' rows in natural order
    if (plan.feasible && workspace_bytes >= plan.bytes) use = B2SP_ALGO_TILE;
    else if (algo == B2SP_ALGO_TILE) return plan.feasible ? B2SP_ERR_WORKSPACE : B2SP_ERR_UNSUPPORTED;
    g_last_algo[B2SP_OP_FUSEDMM] = use;
    int launches = 0;
    g_last_launches[B2SP_OP_FUSEDMM] = 0;
    if (M == 0 || N == 0) return B2SP_OK;
    if (nnz_stride == 0 || Kd == 0) {   // empty patterns or empty dot products: zero outputs
        for (int b = 0; b < batch; ++b) {
            rc = zero_rows(O + (long long)b * stride_o, ldo, M, N, st);
            if (rc != B2SP_OK) return rc;
        }
        return B2SP_OK;
    }
    const long long nz_step = row_ptr_stride == 0 ? 0 : nnz_stride;   // a shared pattern shares its arrays
    const RowBatch rb{row_ptr_stride, nz_step, stride_a, stride_b, stride_d, stride_o};
    if (use == B2SP_ALGO_TILE) {
        BatchDesc bd;
        bd.count = batch; bd.rp = row_ptr_stride; bd.nz = nz_step;
        bd.A = stride_a; bd.B = stride_b; bd.D = stride_d; bd.O = stride_o;
        rc = fused_tile(plan, prepared, 1, M, K, Kd, N, nnz_stride, row_ptr, col_idx, s_values, A, lda, B, ldb, D, ldd,
                        O, ldo, workspace, st, &launches, false, bd, dense_dtype<DT>());
        if (rc != B2SP_OK) return rc;
        int *gate = reinterpret_cast<int *>(static_cast<char *>(workspace) + kWsTileFlagsOffset);
        rc = fused_rows(M, Kd, N, row_ptr, col_idx, s_values, A, lda, B, ldb, D, ldd, O, ldo, nullptr, gate, nullptr, st,
                        batch, rb);
        g_last_launches[B2SP_OP_FUSEDMM] = launches + 1;
        return rc;
    }
    int *clear = reinterpret_cast<int *>(static_cast<char *>(workspace) + kWsStatusOffset);
    rc = fused_rows(M, Kd, N, row_ptr, col_idx, s_values, A, lda, B, ldb, D, ldd, O, ldo, nullptr, nullptr, clear, st,
                    batch, rb);
    g_last_launches[B2SP_OP_FUSEDMM] = 1;
    return rc;
}

extern "C" b2sp_status b2sp_fusedmm_batched(int batch, int M, int K, int Kd, int N, long long nnz_stride,
                                            const int *row_ptr, long long row_ptr_stride, const int *col_idx,
                                            const float *s_values, const float *A, long long lda, long long stride_a,
                                            const float *B, long long ldb, long long stride_b, const float *D,
                                            long long ldd, long long stride_d, float *O, long long ldo,
                                            long long stride_o, void *workspace, size_t workspace_bytes, int algo,
                                            void *stream)
{
    return fusedmm_batched_impl<float>(batch, M, K, Kd, N, nnz_stride, row_ptr, row_ptr_stride, col_idx, s_values, A, lda,
                                       stride_a, B, ldb, stride_b, D, ldd, stride_d, O, ldo, stride_o, workspace,
                                       workspace_bytes, algo, stream);
}
extern "C" b2sp_status b2sp_fusedmm_batched_bf16(int batch, int M, int K, int Kd, int N, long long nnz_stride,
                                                 const int *row_ptr, long long row_ptr_stride, const int *col_idx,
                                                 const float *s_values, const void *A, long long lda, long long stride_a,
                                                 const void *B, long long ldb, long long stride_b, const void *D,
                                                 long long ldd, long long stride_d, float *O, long long ldo,
                                                 long long stride_o, void *workspace, size_t workspace_bytes, int algo,
                                                 void *stream)
{
    return fusedmm_batched_impl<bf16_t>(batch, M, K, Kd, N, nnz_stride, row_ptr, row_ptr_stride, col_idx, s_values,
                                        static_cast<const bf16_t *>(A), lda, stride_a, static_cast<const bf16_t *>(B), ldb,
                                        stride_b, static_cast<const bf16_t *>(D), ldd, stride_d, O, ldo, stride_o,
                                        workspace, workspace_bytes, algo, stream);
}

extern "C" b2sp_status b2sp_prepare_pattern(int M, int K, long long nnz, const int *row_ptr, const int *col_idx,
                                 void *workspace, size_t workspace_bytes, void *stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (bad_csr_args(M, K, nnz, row_ptr, col_idx) || M == 0 || K == 0 || nnz == 0) return B2SP_ERR_INVALID_ARG;
    const size_t need = pattern_table_offset(M) + pattern_table_bytes(M, K);
    b2sp_status rc = check_workspace(workspace, workspace_bytes, need);
    if (rc != B2SP_OK) return rc;
    int launches = 0;
    return pattern_pass(false, M, K, nnz, row_ptr, col_idx, workspace, st, &launches);
}

extern "C" b2sp_status b2sp_validate_csr(int M, int K, long long nnz, const int *row_ptr, const int *col_idx,
                              void *workspace, size_t workspace_bytes, void *stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (M < 0 || K < 0 || nnz < 0 || nnz > (long long)INT_MAX || !row_ptr || (nnz > 0 && !col_idx))
        return B2SP_ERR_INVALID_ARG;
    b2sp_status rc = check_workspace(workspace, workspace_bytes, 256);
    if (rc != B2SP_OK) return rc;
    int *flag = static_cast<int *>(workspace);
    if (cudaMemsetAsync(flag, 0, sizeof(int), st) != cudaSuccess) return B2SP_ERR_CUDA;
    long long work = nnz > M ? nnz : M;
    int blocks = (int)((work + 255) / 256);
    if (blocks < 1) blocks = 1;
    if (blocks > 148 * 16) blocks = 148 * 16;
    validate_csr_kernel<<<blocks, 256, 0, st>>>(M, K, nnz, row_ptr, col_idx, flag);
    if (cudaGetLastError() != cudaSuccess) return B2SP_ERR_CUDA;
    int h = 0;
    if (cudaMemcpyAsync(&h, flag, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return B2SP_ERR_CUDA;
    return h ? B2SP_ERR_BAD_CSR : B2SP_OK;
}

extern "C" b2sp_status b2sp_device_status(const void *workspace, void *stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!workspace) return B2SP_ERR_WORKSPACE;
    int h = 0;
    const int *status = reinterpret_cast<const int *>(static_cast<const char *>(workspace) + 256);
    if (cudaMemcpyAsync(&h, status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return B2SP_ERR_CUDA;
    return h == 0 ? B2SP_OK : B2SP_ERR_TIMEOUT;
}


// ---- host-buffer forms ------------------------------------------------------------------------
namespace {

// Device memory of one host-buffer call.  It comes from a stream-ordered pool that the library owns (one
// per device, created at first use, release threshold "never": freed blocks stay in it across calls, so a
// call does not pay for fresh allocations).  The process's default pool is left as it is.
cudaMemPool_t library_pool()
{
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static cudaMemPool_t pools[kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!pools[dev]) {
        cudaMemPoolProps props = {};
        props.allocType = cudaMemAllocationTypePinned;
        props.handleTypes = cudaMemHandleTypeNone;
        props.location.type = cudaMemLocationTypeDevice;
        props.location.id = dev;
        cudaMemPool_t pool = nullptr;
        if (cudaMemPoolCreate(&pool, &props) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        unsigned long long keep = ~0ull;
        cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &keep);
        pools[dev] = pool;
    }
    return pools[dev];
}

struct DevArena {
    cudaStream_t st;
    cudaMemPool_t pool;
    void *ptrs[16];
    int n = 0;
    bool ok = true;
    int device_word = 0;   // the workspace's status word, copied back with the result
    explicit DevArena(cudaStream_t s) : st(s), pool(library_pool()) { ok = pool != nullptr; }
    void *alloc(size_t bytes)
    {
        void *p = nullptr;
        if (bytes == 0) bytes = 16;
        if (!ok || cudaMallocFromPoolAsync(&p, bytes, pool, st) != cudaSuccess) { ok = false; return nullptr; }
        ptrs[n++] = p;
        return p;
    }
    template <typename T> T *upload(const T *host, size_t count)
    {
        T *d = static_cast<T *>(alloc(sizeof(T) * count));
        if (d && host && count &&
            cudaMemcpyAsync(d, host, sizeof(T) * count, cudaMemcpyHostToDevice, st) != cudaSuccess)
            ok = false;
        return d;
    }
    // Queues the read-back of the status word that device code left in `ws` (a bounded wait that gave up).
    void fetch_status(const void *ws)
    {
        if (ok && ws &&
            cudaMemcpyAsync(&device_word, static_cast<const char *>(ws) + b2sp::kWsStatusOffset, sizeof(int),
                            cudaMemcpyDeviceToHost, st) != cudaSuccess)
            ok = false;
    }
    b2sp_status finish(b2sp_status rc)
    {
        for (int i = 0; i < n; ++i) cudaFreeAsync(ptrs[i], st);
        if (cudaStreamSynchronize(st) != cudaSuccess && rc == B2SP_OK) rc = B2SP_ERR_CUDA;
        if (!ok && rc == B2SP_OK) rc = B2SP_ERR_CUDA;
        if (rc == B2SP_OK && device_word != 0) rc = B2SP_ERR_TIMEOUT;   // the outputs are undefined
        return rc;
    }
};

}  // namespace

extern "C" b2sp_status b2sp_spmm_host(int M, int K, int N, long long nnz, const int *row_ptr,
                           const int *col_idx, const float *values, const float *D, float *O,
                           void *stream)
{
    if (bad_csr_args(M, K, nnz, row_ptr, col_idx) || N < 0) return B2SP_ERR_INVALID_ARG;
    if ((M > 0 && N > 0 && !O) || (nnz > 0 && N > 0 && (!values || !D))) return B2SP_ERR_INVALID_ARG;
    DevArena a(static_cast<cudaStream_t>(stream));
    int *d_rp = a.upload(row_ptr, (size_t)M + 1);
    int *d_ci = a.upload(col_idx, (size_t)nnz);
    float *d_v = a.upload(values, (size_t)nnz);
    float *d_D = a.upload(D, (size_t)K * N);
    float *d_O = static_cast<float *>(a.alloc(sizeof(float) * (size_t)M * N));
    size_t wsb = b2sp_workspace_bytes_algo(B2SP_OP_SPMM, B2SP_ALGO_AUTO, M, K, 0, N, nnz);
    void *ws = a.alloc(wsb);
    b2sp_status rc = B2SP_ERR_CUDA;
    const bool launched_work = M > 0 && N > 0 && nnz > 0;   // otherwise no kernel ran and the status word is unset
    if (a.ok) {
        rc = b2sp_spmm(M, K, N, nnz, d_rp, d_ci, d_v, d_D, N, d_O, N, ws, wsb, B2SP_ALGO_AUTO, stream);
        if (rc == B2SP_OK && (size_t)M * N > 0 &&
            cudaMemcpyAsync(O, d_O, sizeof(float) * (size_t)M * N, cudaMemcpyDeviceToHost, a.st) != cudaSuccess)
            rc = B2SP_ERR_CUDA;
        if (rc == B2SP_OK && launched_work) a.fetch_status(ws);
    }
    return a.finish(rc);
}

extern "C" b2sp_status b2sp_sddmm_host(int M, int K, int Kd, long long nnz, const int *row_ptr,
                            const int *col_idx, const float *s_values, const float *A,
                            const float *B, float *out_values, void *stream)
{
    if (bad_csr_args(M, K, nnz, row_ptr, col_idx) || Kd < 0) return B2SP_ERR_INVALID_ARG;
    if (nnz > 0 && (!out_values || (Kd > 0 && (!A || !B)))) return B2SP_ERR_INVALID_ARG;
    DevArena a(static_cast<cudaStream_t>(stream));
    int *d_rp = a.upload(row_ptr, (size_t)M + 1);
    int *d_ci = a.upload(col_idx, (size_t)nnz);
    float *d_v = s_values ? a.upload(s_values, (size_t)nnz) : nullptr;
    float *d_A = a.upload(A, (size_t)M * Kd);
    float *d_B = a.upload(B, (size_t)K * Kd);
    float *d_C = static_cast<float *>(a.alloc(sizeof(float) * (size_t)nnz));
    size_t wsb = b2sp_workspace_bytes_algo(B2SP_OP_SDDMM, B2SP_ALGO_AUTO, M, K, Kd, 0, nnz);
    void *ws = a.alloc(wsb);
    b2sp_status rc = B2SP_ERR_CUDA;
    const bool launched_work = M > 0 && Kd > 0 && nnz > 0;
    if (a.ok) {
        rc = b2sp_sddmm(M, K, Kd, nnz, d_rp, d_ci, d_v, d_A, Kd, d_B, Kd, d_C, ws, wsb, B2SP_ALGO_AUTO, stream);
        if (rc == B2SP_OK && nnz > 0 &&
            cudaMemcpyAsync(out_values, d_C, sizeof(float) * (size_t)nnz, cudaMemcpyDeviceToHost, a.st) != cudaSuccess)
            rc = B2SP_ERR_CUDA;
        if (rc == B2SP_OK && launched_work) a.fetch_status(ws);
    }
    return a.finish(rc);
}

extern "C" b2sp_status b2sp_fusedmm_host(int M, int K, int Kd, int N, long long nnz, const int *row_ptr,
                              const int *col_idx, const float *s_values, const float *A,
                              const float *B, const float *D, float *O, void *stream)
{
    if (bad_csr_args(M, K, nnz, row_ptr, col_idx) || Kd < 0 || N < 0) return B2SP_ERR_INVALID_ARG;
    if ((M > 0 && N > 0 && !O) || (nnz > 0 && N > 0 && (!D || (Kd > 0 && (!A || !B)))))
        return B2SP_ERR_INVALID_ARG;
    DevArena a(static_cast<cudaStream_t>(stream));
    int *d_rp = a.upload(row_ptr, (size_t)M + 1);
    int *d_ci = a.upload(col_idx, (size_t)nnz);
    float *d_v = s_values ? a.upload(s_values, (size_t)nnz) : nullptr;
    float *d_A = a.upload(A, (size_t)M * Kd);
    float *d_B = a.upload(B, (size_t)K * Kd);
    float *d_D = a.upload(D, (size_t)K * N);
    float *d_O = static_cast<float *>(a.alloc(sizeof(float) * (size_t)M * N));
    size_t wsb = b2sp_workspace_bytes_algo(B2SP_OP_FUSEDMM, B2SP_ALGO_AUTO, M, K, Kd, N, nnz);
    void *ws = a.alloc(wsb);
    b2sp_status rc = B2SP_ERR_CUDA;
    const bool launched_work = M > 0 && N > 0 && Kd > 0 && nnz > 0;
    if (a.ok) {
        rc = b2sp_fusedmm(M, K, Kd, N, nnz, d_rp, d_ci, d_v, d_A, Kd, d_B, Kd, d_D, N, d_O, N, ws, wsb,
                          B2SP_ALGO_AUTO, stream);
        if (rc == B2SP_OK && (size_t)M * N > 0 &&
            cudaMemcpyAsync(O, d_O, sizeof(float) * (size_t)M * N, cudaMemcpyDeviceToHost, a.st) != cudaSuccess)
            rc = B2SP_ERR_CUDA;
        if (rc == B2SP_OK && launched_work) a.fetch_status(ws);
    }
    return a.finish(rc);
}

