"""CPU oracle (fp64) for SPMM / SDDMM / FusedMM -- TEST INFRASTRUCTURE ONLY.

Thin ctypes loader around ``oracle.c`` (built by gcc into ``liboracle.so`` beside it).
Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library and its Python binding never do, and nothing here imports them.

Every function takes numpy arrays (int32 CSR arrays, fp32 dense operands) and returns
``(result, T)`` in float64, where ``T`` is the per-output tolerance scale (sum of |terms|).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None

RTOL = 1e-5   # |x - ref| <= RTOL * T + ATOL
ATOL = 1e-6


def build(force: bool = False) -> str:
    """Compile oracle.c with gcc (-O2 -fopenmp).  Rebuilds when the source is newer."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def _p(a, ct):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def _i32(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a


def _f32(a):
    if a is None:
        return None
    assert a.dtype == np.float32
    return np.ascontiguousarray(a)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def spmm(row_ptr, col_idx, values, D, rows=None):
    """Eq. 2 / Alg. 2.  O = S @ D.  `rows=(r0, r1)` restricts to a row range."""
    lib = _load()
    row_ptr, col_idx, values, D = _i32(row_ptr), _i32(col_idx), _f32(values), _f32(D)
    N = D.shape[1]
    r0, r1 = (0, len(row_ptr) - 1) if rows is None else rows
    O = np.empty((r1 - r0, N), dtype=np.float64)
    T = np.empty_like(O)
    lib.oracle_spmm_rows(ctypes.c_int(r0), ctypes.c_int(r1), ctypes.c_int(N),
                         _p(row_ptr, ctypes.c_int), _p(col_idx, ctypes.c_int),
                         _p(values, ctypes.c_float), _p(D, ctypes.c_float),
                         ctypes.c_longlong(D.shape[1]), _p(O, ctypes.c_double),
                         _p(T, ctypes.c_double))
    return O, T


def sddmm(row_ptr, col_idx, s_values, A, B, rows=None):
    """Eq. 1 / Alg. 1 with value scaling.  C[p] = s_p * <A_i, B_j>; s_values=None => 1."""
    lib = _load()
    row_ptr, col_idx, s_values = _i32(row_ptr), _i32(col_idx), _f32(s_values)
    A, B = _f32(A), _f32(B)
    Kd = A.shape[1]
    assert B.shape[1] == Kd
    r0, r1 = (0, len(row_ptr) - 1) if rows is None else rows
    n = int(row_ptr[r1] - row_ptr[r0])
    C = np.empty(n, dtype=np.float64)
    T = np.empty_like(C)
    lib.oracle_sddmm_rows(ctypes.c_int(r0), ctypes.c_int(r1), ctypes.c_int(Kd),
                          _p(row_ptr, ctypes.c_int), _p(col_idx, ctypes.c_int),
                          _p(s_values, ctypes.c_float), _p(A, ctypes.c_float),
                          ctypes.c_longlong(Kd), _p(B, ctypes.c_float), ctypes.c_longlong(Kd),
                          _p(C, ctypes.c_double), _p(T, ctypes.c_double))
    return C, T


def fusedmm(row_ptr, col_idx, s_values, A, B, D, rows=None):
    """Eq. 3 / Alg. 3.  O = (S .* (A @ B.T)) @ D without rounding the sampled values."""
    lib = _load()
    row_ptr, col_idx, s_values = _i32(row_ptr), _i32(col_idx), _f32(s_values)
    A, B, D = _f32(A), _f32(B), _f32(D)
    Kd, N = A.shape[1], D.shape[1]
    assert B.shape[1] == Kd and B.shape[0] == D.shape[0]
    r0, r1 = (0, len(row_ptr) - 1) if rows is None else rows
    O = np.empty((r1 - r0, N), dtype=np.float64)
    T = np.empty_like(O)
    lib.oracle_fusedmm_rows(ctypes.c_int(r0), ctypes.c_int(r1), ctypes.c_int(Kd),
                            ctypes.c_int(N), _p(row_ptr, ctypes.c_int),
                            _p(col_idx, ctypes.c_int), _p(s_values, ctypes.c_float),
                            _p(A, ctypes.c_float), ctypes.c_longlong(Kd),
                            _p(B, ctypes.c_float), ctypes.c_longlong(Kd),
                            _p(D, ctypes.c_float), ctypes.c_longlong(N),
                            _p(O, ctypes.c_double), _p(T, ctypes.c_double))
    return O, T


def within_tolerance(x, ref, T, rtol: float = RTOL, atol: float = ATOL):
    """Elementwise gate |x - ref| <= rtol*T + atol.  Returns (ok, worst ratio err/bound)."""
    x = np.asarray(x, dtype=np.float64)
    err = np.abs(x - ref)
    bound = rtol * T + atol
    ratio = float((err / bound).max()) if err.size else 0.0
    return bool(np.all(err <= bound)) and bool(np.all(np.isfinite(x))), ratio
