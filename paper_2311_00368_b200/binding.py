"""Thin Python binding over the C-ABI library ``libb2sp.so``: argument marshalling only.

Every step of the three ops runs inside the CUDA library; this module turns torch tensors
into raw device pointers + sizes, supplies a workspace and the current CUDA stream, and
raises on a non-zero status.  There is no CPU fallback: importing this module raises
``ImportError`` if the library has not been built, and calling an op without a CUDA device
fails in the library.

Function names and argument order follow ``include/b2sp.h`` (and ``include/b2sp_debug.h``).
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("B2SP_LIB") or os.path.join(_HERE, "libb2sp.so")  # B2SP_LIB: alternate build

ALGO_AUTO, ALGO_ROW, ALGO_ROW_NAT, ALGO_TILE, ALGO_TILE_PREPARED = 0, 1, 2, 3, 4
OP_SPMM, OP_SDDMM, OP_FUSEDMM = 0, 1, 2
ALGO_NAMES = {0: "auto", 1: "row", 2: "row_nat", 3: "tile", 4: "tile_prepared", -1: "none"}

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2311_00368_b200.build` "
        "(there is no fallback implementation)")

lib = ctypes.CDLL(LIB_PATH)

_i, _ll, _vp, _sz = ctypes.c_int, ctypes.c_longlong, ctypes.c_void_p, ctypes.c_size_t

lib.b2sp_version.restype = _i
lib.b2sp_status_string.restype = ctypes.c_char_p
lib.b2sp_status_string.argtypes = [_i]
lib.b2sp_workspace_bytes.restype = _sz
lib.b2sp_workspace_bytes.argtypes = [_i, _i, _i, _i, _i, _ll]
lib.b2sp_workspace_bytes_algo.restype = _sz
lib.b2sp_workspace_bytes_algo.argtypes = [_i, _i, _i, _i, _i, _i, _ll]
lib.b2sp_spmm.restype = _i
lib.b2sp_spmm.argtypes = [_i, _i, _i, _ll, _vp, _vp, _vp, _vp, _ll, _vp, _ll, _vp, _sz, _i, _vp]
lib.b2sp_sddmm.restype = _i
lib.b2sp_sddmm.argtypes = [_i, _i, _i, _ll, _vp, _vp, _vp, _vp, _ll, _vp, _ll, _vp, _vp, _sz, _i, _vp]
lib.b2sp_fusedmm.restype = _i
lib.b2sp_fusedmm.argtypes = [_i, _i, _i, _i, _ll, _vp, _vp, _vp, _vp, _ll, _vp, _ll, _vp, _ll, _vp, _ll,
                             _vp, _sz, _i, _vp]
lib.b2sp_spmm_bf16.restype = _i
lib.b2sp_spmm_bf16.argtypes = lib.b2sp_spmm.argtypes
lib.b2sp_sddmm_bf16.restype = _i
lib.b2sp_sddmm_bf16.argtypes = lib.b2sp_sddmm.argtypes
lib.b2sp_fusedmm_bf16.restype = _i
lib.b2sp_fusedmm_bf16.argtypes = lib.b2sp_fusedmm.argtypes
lib.b2sp_spmm_host.restype = _i
lib.b2sp_spmm_host.argtypes = [_i, _i, _i, _ll, _vp, _vp, _vp, _vp, _vp, _vp]
lib.b2sp_sddmm_host.restype = _i
lib.b2sp_sddmm_host.argtypes = [_i, _i, _i, _ll, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
lib.b2sp_fusedmm_host.restype = _i
lib.b2sp_fusedmm_host.argtypes = [_i, _i, _i, _i, _ll, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
lib.b2sp_spmm_static_scratch.restype = _i
lib.b2sp_spmm_static_scratch.argtypes = [_i, _i, _i, _ll, _vp, _vp, _vp, _vp, _ll, _vp, _ll, _vp]
lib.b2sp_workspace_bytes_batched.restype = _sz
lib.b2sp_workspace_bytes_batched.argtypes = [_i, _i, _i, _i, _i, _ll]
lib.b2sp_prepare_pattern_batched.restype = _i
lib.b2sp_prepare_pattern_batched.argtypes = [_i, _i, _i, _ll, _vp, _ll, _vp, _vp, _sz, _vp]
lib.b2sp_fusedmm_batched.restype = _i
lib.b2sp_fusedmm_batched.argtypes = [_i, _i, _i, _i, _i, _ll, _vp, _ll, _vp, _vp, _vp, _ll, _ll, _vp, _ll, _ll,
                                     _vp, _ll, _ll, _vp, _ll, _ll, _vp, _sz, _i, _vp]
lib.b2sp_fusedmm_batched_bf16.restype = _i
lib.b2sp_fusedmm_batched_bf16.argtypes = lib.b2sp_fusedmm_batched.argtypes
lib.b2sp_prepare_pattern.restype = _i
lib.b2sp_prepare_pattern.argtypes = [_i, _i, _ll, _vp, _vp, _vp, _sz, _vp]
lib.b2sp_validate_csr.restype = _i
lib.b2sp_validate_csr.argtypes = [_i, _i, _ll, _vp, _vp, _vp, _sz, _vp]
lib.b2sp_probe_fp32_peak.restype = _i
lib.b2sp_probe_fp32_peak.argtypes = [_i, _vp, ctypes.POINTER(ctypes.c_double), _vp]
lib.b2sp_probe_l2_pull.restype = _i
lib.b2sp_probe_l2_pull.argtypes = [_vp, ctypes.c_size_t, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double), _vp]
lib.b2sp_device_status.restype = _i
lib.b2sp_device_status.argtypes = [_vp, _vp]
lib.b2sp_last_algo.restype = _i
lib.b2sp_last_algo.argtypes = [_i]
lib.b2sp_last_launches.restype = _i
lib.b2sp_last_launches.argtypes = [_i]
lib.b2sp_debug_force_k_splits.restype = None
lib.b2sp_debug_force_k_splits.argtypes = [_i]
lib.b2sp_debug_force_partition.restype = None
lib.b2sp_debug_force_partition.argtypes = [_i]
lib.b2sp_debug_inject_wait_timeout.restype = _i
lib.b2sp_debug_inject_wait_timeout.argtypes = [_i, ctypes.c_ulonglong]


class B2spError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib.b2sp_status_string(status).decode()} (status {status})")


def _check(status: int, where: str):
    if status != 0:
        raise B2spError(status, where)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ld(t):
    assert t.dim() == 2 and (t.shape[1] <= 1 or t.stride(1) == 1), "dense operands are row-major"
    return t.stride(0) if t.shape[0] > 1 else max(t.shape[1], t.stride(0))


def _want(t, dtype, name, cuda=True):
    if t is None:
        return
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}")
    if cuda and not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")


def version() -> int:
    return int(lib.b2sp_version())


def workspace_bytes(op: int, M: int, K: int, Kd: int, N: int, nnz: int, algo=None) -> int:
    """b2sp_workspace_bytes (upper bound over all algo values) or, with `algo`, b2sp_workspace_bytes_algo."""
    if algo is None:
        return int(lib.b2sp_workspace_bytes(op, M, K, Kd, N, nnz))
    return int(lib.b2sp_workspace_bytes_algo(op, algo, M, K, Kd, N, nnz))


_ws_cache = {}


def _workspace(op, M, K, Kd, N, nnz, device, workspace, algo=0):
    if workspace is None:
        need = workspace_bytes(op, M, K, Kd, N, nnz, algo)
        key = (device.index, torch.cuda.current_stream(device).cuda_stream)
        workspace = _ws_cache.get(key)
        if workspace is None or workspace.numel() < need:
            workspace = torch.empty(max(need, 1 << 20), dtype=torch.uint8, device=device)
            _ws_cache[key] = workspace
    return workspace, workspace.numel()


def probe_fp32_peak(iters: int = 4096, device=None) -> float:
    """b2sp_probe_fp32_peak: sustained FP32 FMA rate of the current device in GFLOP/s (synchronises)."""
    scratch = torch.zeros(1, dtype=torch.float32, device=device or "cuda")
    out = ctypes.c_double(0.0)
    _check(lib.b2sp_probe_fp32_peak(iters, _ptr(scratch), ctypes.byref(out), _stream()), "b2sp_probe_fp32_peak")
    return float(out.value)


def probe_l2_pull(device=None):
    """b2sp_probe_l2_pull: (GB/s per SM, GB/s of the whole GPU) of 32 KB bulk copies from L2 into shared memory (synchronises)."""
    scratch = torch.zeros((17 << 20) + 64, dtype=torch.uint8, device=device or "cuda")
    per_sm, total = ctypes.c_double(0.0), ctypes.c_double(0.0)
    _check(lib.b2sp_probe_l2_pull(_ptr(scratch), scratch.numel(), ctypes.byref(per_sm), ctypes.byref(total), _stream()),
           "b2sp_probe_l2_pull")
    return float(per_sm.value), float(total.value)


def last_algo(op: int) -> int:
    return int(lib.b2sp_last_algo(op))


def last_launches(op: int) -> int:
    return int(lib.b2sp_last_launches(op))


def debug_force_k_splits(k_splits: int) -> None:
    """b2sp_debug_force_k_splits: override the dense-tile planner's K split (0 = planner's choice)."""
    lib.b2sp_debug_force_k_splits(int(k_splits))


def debug_force_partition(partition: int) -> None:
    """b2sp_debug_force_partition: 0 = planner's choice, 1 = tiles x K splits only, 2 = balanced wherever offered."""
    lib.b2sp_debug_force_partition(int(partition))


def debug_inject_wait_timeout(chunk: int, limit_ns: int = 0) -> None:
    """b2sp_debug_inject_wait_timeout: make the dense-tile kernels' bounded waits run out (chunk >= 0) with a
    short limit, or switch the hook off again (chunk < 0)."""
    _check(lib.b2sp_debug_inject_wait_timeout(int(chunk), int(limit_ns)), "b2sp_debug_inject_wait_timeout")


def spmm(row_ptr, col_idx, values, D, K=None, out=None, workspace=None, algo=ALGO_AUTO, dtype=torch.float32):
    """b2sp_spmm: O = S @ D.  CSR tensors int32/fp32 on the GPU; D [K, N] fp32 row-major
    (dtype=torch.bfloat16: b2sp_spmm_bf16, D in bfloat16)."""
    _want(row_ptr, torch.int32, "row_ptr"); _want(col_idx, torch.int32, "col_idx")
    _want(values, torch.float32, "values"); _want(D, dtype, "D")
    M, nnz = row_ptr.numel() - 1, col_idx.numel()
    K = D.shape[0] if K is None else K
    N = D.shape[1]
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32, device=D.device)
    ws, wsb = _workspace(OP_SPMM, M, K, 0, N, nnz, D.device, workspace, algo)
    fn, name = (lib.b2sp_spmm, "b2sp_spmm") if dtype == torch.float32 else (lib.b2sp_spmm_bf16, "b2sp_spmm_bf16")
    _check(fn(M, K, N, nnz, _ptr(row_ptr), _ptr(col_idx), _ptr(values), _ptr(D), _ld(D),
                         _ptr(out), _ld(out), _ptr(ws), wsb, algo, _stream()), name)
    return out


STATIC_SCRATCH_MAX_ROWS = 65536


def spmm_static_scratch(row_ptr, col_idx, values, D, K=None, out=None):
    """b2sp_spmm_static_scratch: SPMM for callers that may not allocate device memory.  The
    library's built-in scratch array replaces the workspace; M is limited to
    STATIC_SCRATCH_MAX_ROWS, and calls that could overlap on the GPU must not share a device.
    (`out` should be passed by such callers; it is only created here for convenience.)"""
    _want(row_ptr, torch.int32, "row_ptr"); _want(col_idx, torch.int32, "col_idx")
    _want(values, torch.float32, "values"); _want(D, torch.float32, "D")
    M, nnz = row_ptr.numel() - 1, col_idx.numel()
    K = D.shape[0] if K is None else K
    N = D.shape[1]
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32, device=D.device)
    _check(lib.b2sp_spmm_static_scratch(M, K, N, nnz, _ptr(row_ptr), _ptr(col_idx), _ptr(values),
                                        _ptr(D), _ld(D), _ptr(out), _ld(out), _stream()),
           "b2sp_spmm_static_scratch")
    return out


def sddmm(row_ptr, col_idx, s_values, A, B, out=None, workspace=None, algo=ALGO_AUTO, dtype=torch.float32):
    """b2sp_sddmm: out[p] = s_p * <A[i], B[j]> on S's pattern; s_values=None means all ones
    (dtype=torch.bfloat16: b2sp_sddmm_bf16, A and B in bfloat16)."""
    _want(row_ptr, torch.int32, "row_ptr"); _want(col_idx, torch.int32, "col_idx")
    _want(s_values, torch.float32, "s_values"); _want(A, dtype, "A"); _want(B, dtype, "B")
    M, nnz = row_ptr.numel() - 1, col_idx.numel()
    K, Kd = B.shape
    if A.shape != (M, Kd):
        raise ValueError("A must be [M, Kd]")
    if out is None:
        out = torch.empty(nnz, dtype=torch.float32, device=A.device)
    ws, wsb = _workspace(OP_SDDMM, M, K, Kd, 0, nnz, A.device, workspace, algo)
    fn, name = (lib.b2sp_sddmm, "b2sp_sddmm") if dtype == torch.float32 else (lib.b2sp_sddmm_bf16, "b2sp_sddmm_bf16")
    _check(fn(M, K, Kd, nnz, _ptr(row_ptr), _ptr(col_idx), _ptr(s_values), _ptr(A), _ld(A),
                          _ptr(B), _ld(B), _ptr(out), _ptr(ws), wsb, algo, _stream()), name)
    return out


def fusedmm(row_ptr, col_idx, s_values, A, B, D, out=None, workspace=None, algo=ALGO_AUTO, dtype=torch.float32):
    """b2sp_fusedmm: O = (S .* (A @ B.T)) @ D in one pass; the sampled values never reach HBM
    (dtype=torch.bfloat16: b2sp_fusedmm_bf16, A, B and D in bfloat16)."""
    _want(row_ptr, torch.int32, "row_ptr"); _want(col_idx, torch.int32, "col_idx")
    _want(s_values, torch.float32, "s_values"); _want(A, dtype, "A"); _want(B, dtype, "B")
    _want(D, dtype, "D")
    M, nnz = row_ptr.numel() - 1, col_idx.numel()
    K, Kd = B.shape
    N = D.shape[1]
    if A.shape != (M, Kd) or D.shape[0] != K:
        raise ValueError("A must be [M, Kd] and D [K, N]")
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32, device=D.device)
    ws, wsb = _workspace(OP_FUSEDMM, M, K, Kd, N, nnz, D.device, workspace, algo)
    fn, name = (lib.b2sp_fusedmm, "b2sp_fusedmm") if dtype == torch.float32 else (lib.b2sp_fusedmm_bf16, "b2sp_fusedmm_bf16")
    _check(fn(M, K, Kd, N, nnz, _ptr(row_ptr), _ptr(col_idx), _ptr(s_values), _ptr(A),
                            _ld(A), _ptr(B), _ld(B), _ptr(D), _ld(D), _ptr(out), _ld(out), _ptr(ws), wsb,
                            algo, _stream()), name)
    return out


def _batch_dims(row_ptr, col_idx):
    """[batch, M + 1] row pointers and [batch, nnz_stride] column indices (a 1-D row_ptr: one shared pattern)."""
    if row_ptr.dim() == 1:
        return None, row_ptr.numel() - 1, 0, col_idx.shape[-1]
    assert row_ptr.stride(1) == 1 and col_idx.dim() == 2 and col_idx.stride(1) == 1
    return row_ptr.shape[0], row_ptr.shape[1] - 1, row_ptr.stride(0), col_idx.stride(0)


def _batch_stride(t, batch):
    """Element stride between the problems of a [batch, rows, cols] operand (0 for a shared [rows, cols] one)."""
    if t.dim() == 2:
        return 0
    assert t.dim() == 3 and t.shape[0] == batch and (t.shape[2] <= 1 or t.stride(2) == 1)
    return t.stride(0)


def workspace_bytes_batched(batch: int, M: int, K: int, Kd: int, N: int, nnz_stride: int) -> int:
    return int(lib.b2sp_workspace_bytes_batched(batch, M, K, Kd, N, nnz_stride))


def prepare_pattern_batched(row_ptr, col_idx, K, workspace, batch=None):
    """b2sp_prepare_pattern_batched: the window tables of a batch of patterns (row_ptr [batch, M + 1],
    col_idx [batch, nnz_stride]; 1-D tensors with `batch`: one pattern shared by all problems)."""
    nb, M, rps, nzs = _batch_dims(row_ptr, col_idx)
    nb = batch if nb is None else nb
    _check(lib.b2sp_prepare_pattern_batched(nb, M, K, nzs, _ptr(row_ptr), rps, _ptr(col_idx), _ptr(workspace),
                                            workspace.numel(), _stream()), "b2sp_prepare_pattern_batched")


def fusedmm_batched(row_ptr, col_idx, s_values, A, B, D, out=None, workspace=None, algo=ALGO_AUTO, dtype=torch.float32):
    """b2sp_fusedmm_batched: O[b] = (S[b] .* (A[b] @ B[b].T)) @ D[b] for all problems of a batch in one
    call.  row_ptr [batch, M + 1] (each problem's positions start at 0), col_idx / s_values
    [batch, nnz_stride] (rows padded to a common length), A [batch, M, Kd], B [batch, K, Kd],
    D [batch, K, N]; a 1-D row_ptr / col_idx / s_values or a 2-D dense operand is shared by all problems.
    dtype=torch.bfloat16: b2sp_fusedmm_batched_bf16 (A, B, D in bfloat16)."""
    _want(row_ptr, torch.int32, "row_ptr"); _want(col_idx, torch.int32, "col_idx")
    _want(s_values, torch.float32, "s_values"); _want(A, dtype, "A"); _want(B, dtype, "B")
    _want(D, dtype, "D")
    nb, M, rps, nzs = _batch_dims(row_ptr, col_idx)
    if nb is None:
        nb = max(t.shape[0] if t.dim() == 3 else 1 for t in (A, B, D))
    K, Kd, N = B.shape[-2], B.shape[-1], D.shape[-1]
    if out is None:
        out = torch.empty((nb, M, N), dtype=torch.float32, device=D.device)
    assert out.dim() == 3 and out.shape[0] == nb and out.stride(2) == 1
    if workspace is None:
        workspace = torch.empty(max(workspace_bytes_batched(nb, M, K, Kd, N, nzs), 1 << 20), dtype=torch.uint8,
                                device=D.device)
    ld = lambda t: t.stride(-2) if t.shape[-2] > 1 else max(t.shape[-1], t.stride(-2))
    fn, name = ((lib.b2sp_fusedmm_batched, "b2sp_fusedmm_batched") if dtype == torch.float32
                else (lib.b2sp_fusedmm_batched_bf16, "b2sp_fusedmm_batched_bf16"))
    _check(fn(nb, M, K, Kd, N, nzs, _ptr(row_ptr), rps, _ptr(col_idx), _ptr(s_values),
                                    _ptr(A), ld(A), _batch_stride(A, nb), _ptr(B), ld(B), _batch_stride(B, nb),
                                    _ptr(D), ld(D), _batch_stride(D, nb), _ptr(out), ld(out), out.stride(0),
                                    _ptr(workspace), workspace.numel(), algo, _stream()), name)
    return out


def _host(t, dtype, name):
    if t is None:
        return None
    if t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CPU tensor of {dtype}")
    return t


def spmm_host(row_ptr, col_idx, values, D, out):
    """b2sp_spmm_host: host tensors in, host tensor out (copies happen inside the library)."""
    for t, dt, n in ((row_ptr, torch.int32, "row_ptr"), (col_idx, torch.int32, "col_idx"),
                     (values, torch.float32, "values"), (D, torch.float32, "D"), (out, torch.float32, "out")):
        _host(t, dt, n)
    M, nnz = row_ptr.numel() - 1, col_idx.numel()
    K, N = D.shape
    _check(lib.b2sp_spmm_host(M, K, N, nnz, _ptr(row_ptr), _ptr(col_idx), _ptr(values), _ptr(D),
                              _ptr(out), _stream()), "b2sp_spmm_host")
    return out


def sddmm_host(row_ptr, col_idx, s_values, A, B, out):
    for t, dt, n in ((row_ptr, torch.int32, "row_ptr"), (col_idx, torch.int32, "col_idx"),
                     (s_values, torch.float32, "s_values"), (A, torch.float32, "A"),
                     (B, torch.float32, "B"), (out, torch.float32, "out")):
        _host(t, dt, n)
    M, nnz = row_ptr.numel() - 1, col_idx.numel()
    K, Kd = B.shape
    _check(lib.b2sp_sddmm_host(M, K, Kd, nnz, _ptr(row_ptr), _ptr(col_idx), _ptr(s_values), _ptr(A),
                               _ptr(B), _ptr(out), _stream()), "b2sp_sddmm_host")
    return out


def fusedmm_host(row_ptr, col_idx, s_values, A, B, D, out):
    for t, dt, n in ((row_ptr, torch.int32, "row_ptr"), (col_idx, torch.int32, "col_idx"),
                     (s_values, torch.float32, "s_values"), (A, torch.float32, "A"),
                     (B, torch.float32, "B"), (D, torch.float32, "D"), (out, torch.float32, "out")):
        _host(t, dt, n)
    M, nnz = row_ptr.numel() - 1, col_idx.numel()
    K, Kd = B.shape
    N = D.shape[1]
    _check(lib.b2sp_fusedmm_host(M, K, Kd, N, nnz, _ptr(row_ptr), _ptr(col_idx), _ptr(s_values),
                                 _ptr(A), _ptr(B), _ptr(D), _ptr(out), _stream()), "b2sp_fusedmm_host")
    return out


def prepare_pattern(row_ptr, col_idx, K, workspace):
    """b2sp_prepare_pattern: build S's window table in `workspace` once; later calls that pass the same
    workspace and algo=ALGO_TILE_PREPARED reuse it."""
    M, nnz = row_ptr.numel() - 1, col_idx.numel()
    _check(lib.b2sp_prepare_pattern(M, K, nnz, _ptr(row_ptr), _ptr(col_idx), _ptr(workspace),
                                    workspace.numel(), _stream()), "b2sp_prepare_pattern")


def validate_csr(row_ptr, col_idx, K) -> bool:
    """b2sp_validate_csr: True if the CSR arrays are well formed (synchronises)."""
    M, nnz = row_ptr.numel() - 1, col_idx.numel()
    ws = torch.empty(256, dtype=torch.uint8, device=row_ptr.device)
    st = lib.b2sp_validate_csr(M, K, nnz, _ptr(row_ptr), _ptr(col_idx), _ptr(ws), 256, _stream())
    if st == 3:
        return False
    _check(st, "b2sp_validate_csr")
    return True


def device_status(workspace) -> int:
    return int(lib.b2sp_device_status(_ptr(workspace), _stream()))
