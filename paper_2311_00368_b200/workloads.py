"""Seeded synthetic inputs for SPMM / SDDMM / FusedMM.

This module only *draws inputs*: CSR sparsity patterns, their values and the dense
operands.  It holds none of the arithmetic of the three operations, so both the CPU
oracle's tests and the CUDA path's tests/bench may import it.

Layout follows the paper's storage section: CSR with 0-based int32 ``row_ptr`` (M+1),
``col_idx`` (nnz), fp32 ``values`` (nnz), rows in order, columns sorted and unique
within a row; dense operands fp32 row-major.

Generator: ``numpy.random.default_rng(seed)`` (PCG64).  Draw order per problem:
pattern, S values, A, B, D.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np

_BLOCK_ROWS = 1024


@dataclass
class Problem:
    """One (S, A, B, D) instance.  Any of A/B/D may be None when an op does not use it."""

    name: str
    M: int
    K: int
    row_ptr: np.ndarray  # int32 [M+1]
    col_idx: np.ndarray  # int32 [nnz]
    values: np.ndarray  # float32 [nnz]
    Kd: int = 0
    N: int = 0
    A: Optional[np.ndarray] = None  # float32 [M, Kd]
    B: Optional[np.ndarray] = None  # float32 [K, Kd]
    D: Optional[np.ndarray] = None  # float32 [K, N]

    @property
    def nnz(self) -> int:
        return int(self.row_ptr[-1])


# ----------------------------------------------------------------------------------
# patterns
# ----------------------------------------------------------------------------------

def _rows_to_csr(row_cols: list, M: int) -> tuple:
    lens = np.fromiter((len(c) for c in row_cols), dtype=np.int64, count=M)
    row_ptr = np.zeros(M + 1, dtype=np.int64)
    np.cumsum(lens, out=row_ptr[1:])
    assert row_ptr[-1] < 2**31
    col_idx = np.concatenate(row_cols).astype(np.int32) if M else np.zeros(0, np.int32)
    return row_ptr.astype(np.int32), col_idx


def _mask_to_csr(mask_blocks, M: int) -> tuple:
    """mask_blocks yields (row0, bool[rows, K]) in row order."""
    counts = np.zeros(M, dtype=np.int64)
    cols = []
    for r0, mask in mask_blocks:
        counts[r0:r0 + mask.shape[0]] = mask.sum(axis=1)
        cols.append(np.nonzero(mask)[1].astype(np.int32))  # row-major order => sorted in-row
    row_ptr = np.zeros(M + 1, dtype=np.int64)
    np.cumsum(counts, out=row_ptr[1:])
    assert row_ptr[-1] < 2**31
    col_idx = np.concatenate(cols) if cols else np.zeros(0, np.int32)
    return row_ptr.astype(np.int32), col_idx


def pattern_uniform(rng, M: int, K: int, density: float) -> tuple:
    """Independent Bernoulli(density) per entry, drawn in blocks of 1024 rows."""

    def blocks():
        for r0 in range(0, M, _BLOCK_ROWS):
            rows = min(_BLOCK_ROWS, M - r0)
            yield r0, rng.random((rows, K), dtype=np.float32) < np.float32(density)

    return _mask_to_csr(blocks(), M)


def band_entry_count(M: int, K: int, half: int) -> int:
    i = np.arange(M, dtype=np.int64)
    lo = np.clip(i - half, 0, K)
    hi = np.clip(i + half, 0, K)
    return int((hi - lo).sum())


def pattern_band_plus_uniform(rng, M: int, K: int, band: int, density: float) -> tuple:
    """A `band`-wide diagonal band j in [i-band/2, i+band/2) clipped to the matrix, united
    with Bernoulli(p) on every other position, p chosen so the expected total density is
    `density` (sparse-attention shaped: local window + random global links)."""
    half = band // 2
    nband = band_entry_count(M, K, half)
    p = (density * M * K - nband) / float(M * K - nband)
    assert 0.0 <= p <= 1.0

    def blocks():
        j = np.arange(K, dtype=np.int64)[None, :]
        for r0 in range(0, M, _BLOCK_ROWS):
            rows = min(_BLOCK_ROWS, M - r0)
            i = np.arange(r0, r0 + rows, dtype=np.int64)[:, None]
            in_band = (j >= i - half) & (j < i + half)
            extra = rng.random((rows, K), dtype=np.float32) < np.float32(p)
            yield r0, in_band | extra

    return _mask_to_csr(blocks(), M)


def powerlaw_row_lengths(M: int, K: int, density: float, exponent: float = 1.1) -> np.ndarray:
    """Deterministic Zipf-shaped row lengths by rank r = 1..M: len(r) = min(K, c * r**-exponent)
    with c found by bisection so that the lengths sum to round(density*M*K); fractional parts
    are distributed by largest remainder so the total is exact."""
    target = int(round(density * M * K))
    r = np.arange(1, M + 1, dtype=np.float64)
    w = r ** (-exponent)

    def total(c):
        return np.minimum(float(K), c * w).sum()

    lo, hi = 0.0, float(K) / w[-1]
    assert total(hi) >= target
    for _ in range(200):
        mid = 0.5 * (lo + hi)
        if total(mid) < target:
            lo = mid
        else:
            hi = mid
    real = np.minimum(float(K), hi * w)
    base = np.floor(real).astype(np.int64)
    deficit = target - int(base.sum())
    if deficit > 0:
        frac = real - base
        frac[base >= K] = -1.0
        order = np.argsort(-frac, kind="stable")
        base[order[:deficit]] += 1
    elif deficit < 0:
        frac = real - base
        order = np.argsort(frac, kind="stable")
        order = order[base[order] > 0]
        base[order[:-deficit]] -= 1
    assert int(base.sum()) == target and base.max() <= K and base.min() >= 0
    return base


def pattern_powerlaw(rng, M: int, K: int, density: float, exponent: float = 1.1,
                     shuffle: bool = True) -> tuple:
    """Power-law row lengths (see powerlaw_row_lengths), ranks assigned to rows by a random
    permutation; each row's columns are a uniform random subset of that size, sorted."""
    lens_by_rank = powerlaw_row_lengths(M, K, density, exponent)
    perm = rng.permutation(M) if shuffle else np.arange(M)
    lens = np.empty(M, dtype=np.int64)
    lens[perm] = lens_by_rank
    row_cols = []
    for r0 in range(0, M, _BLOCK_ROWS):
        rows = min(_BLOCK_ROWS, M - r0)
        order = np.argsort(rng.random((rows, K), dtype=np.float32), axis=1, kind="stable")
        for t in range(rows):
            row_cols.append(np.sort(order[t, :lens[r0 + t]]).astype(np.int32))
    return _rows_to_csr(row_cols, M)


# ----------------------------------------------------------------------------------
# values and dense operands
# ----------------------------------------------------------------------------------

def values_uniform(rng, nnz: int) -> np.ndarray:
    return rng.uniform(-1.0, 1.0, nnz).astype(np.float32)


def values_ones(nnz: int) -> np.ndarray:
    return np.ones(nnz, dtype=np.float32)


def dense_normal(rng, rows: int, cols: int) -> np.ndarray:
    return rng.standard_normal((rows, cols), dtype=np.float32)


def _finish(name, rng, M, K, row_ptr, col_idx, unit_values, Kd, N) -> Problem:
    nnz = int(row_ptr[-1])
    values = values_ones(nnz) if unit_values else values_uniform(rng, nnz)
    A = dense_normal(rng, M, Kd) if Kd else None
    B = dense_normal(rng, K, Kd) if Kd else None
    D = dense_normal(rng, K, N) if N else None
    return Problem(name, M, K, row_ptr, col_idx, values, Kd, N, A, B, D)


# ----------------------------------------------------------------------------------
# the five named workloads
# ----------------------------------------------------------------------------------

def tiny(seed: int = 0) -> Problem:
    """256x256, 10% uniform, values U(-1,1); A,B 256x64; D 256x64."""
    rng = np.random.default_rng(seed)
    rp, ci = pattern_uniform(rng, 256, 256, 0.10)
    return _finish("tiny", rng, 256, 256, rp, ci, False, 64, 64)


def spmm_case(seed: int = 1, M: int = 2048, K: int = 2048, density: float = 0.20,
              N: int = 256) -> Problem:
    """2048x2048, 20% uniform, values U(-1,1); D 2048x256."""
    rng = np.random.default_rng(seed)
    rp, ci = pattern_uniform(rng, M, K, density)
    return _finish("spmm", rng, M, K, rp, ci, False, 0, N)


def sddmm_case(seed: int = 2, M: int = 4096, K: int = 4096, density: float = 0.10,
               Kd: int = 128) -> Problem:
    """4096x4096, 10% uniform, values all 1.0; A,B 4096x128."""
    rng = np.random.default_rng(seed)
    rp, ci = pattern_uniform(rng, M, K, density)
    return _finish("sddmm", rng, M, K, rp, ci, True, Kd, 0)


def attention_case(problem: int, seed: int = 3, L: int = 4096, head_dim: int = 64,
                   band: int = 128, density: float = 0.20) -> Problem:
    """One of the independent (batch x head) problems: band + uniform extras, values 1.0;
    Q=A, K=B, V=D are L x head_dim.  Per-problem generator default_rng([seed, problem])."""
    rng = np.random.default_rng([seed, problem])
    rp, ci = pattern_band_plus_uniform(rng, L, L, band, density)
    return _finish(f"attn{problem}", rng, L, L, rp, ci, True, head_dim, head_dim)


def sweep_case(density: float, N: int, seed: int = 4, M: int = 8192, K: int = 8192,
               Kd: int = 128, shuffle: bool = True) -> Problem:
    """8192x8192 power-law rows (Zipf exponent 1.1) at the given mean density, values
    U(-1,1); A,B 8192xKd; D 8192xN."""
    rng = np.random.default_rng(seed)
    rp, ci = pattern_powerlaw(rng, M, K, density, 1.1, shuffle)
    return _finish(f"sweep_d{int(round(density * 100))}_n{N}", rng, M, K, rp, ci, False, Kd, N)


# The paper's evaluation grid (the x axis of its benchmark figures): 12 shapes x N in {32, 128} x
# sparsity in {70, 80, 90}%.  Its matrices (a public collection) are not available here; these are
# uniform-random stand-ins of the same shape and density.  "1k" is read as 1024.
PAPER_GRID_SHAPES = [(1, 1), (3, 1), (4, 1), (2, 2), (6, 2), (8, 2), (4, 4), (12, 4), (16, 4), (8, 8), (24, 8), (32, 8)]
PAPER_GRID_WIDTHS = (32, 128)
PAPER_GRID_SPARSITIES = (70, 80, 90)


def paper_grid_names() -> list:
    """Names of the 72 grid cases, in the order of the paper's figures (N = 32 first)."""
    return [f"grid_{m}k_{k}k_{n}_{sp}" for n in PAPER_GRID_WIDTHS for (m, k) in PAPER_GRID_SHAPES
            for sp in PAPER_GRID_SPARSITIES]


def paper_grid_case(name: str, seed: int = 5) -> Problem:
    """`grid_<M>k_<K>k_<N>_<sparsity%>`: S is M x K uniform-random at density 1 - sparsity with values
    U(-1,1); A is M x N, B and D are K x N (the paper uses one width N for the dot product and for
    the output).  The generator is seeded by (seed, M, K, N, sparsity)."""
    _, m, k, n, sp = name.split("_")
    M, K, N, sp = int(m[:-1]) * 1024, int(k[:-1]) * 1024, int(n), int(sp)
    rng = np.random.default_rng([seed, M, K, N, sp])
    rp, ci = pattern_uniform(rng, M, K, 1.0 - sp / 100.0)
    return _finish(name, rng, M, K, rp, ci, False, N, N)


def small_random(seed: int, M: int, K: int, density: float, Kd: int, N: int,
                 unit_values: bool = False, kind: str = "uniform") -> Problem:
    """Arbitrary small instance for parity and edge-case tests."""
    rng = np.random.default_rng(seed)
    if kind == "uniform":
        rp, ci = pattern_uniform(rng, M, K, density)
    elif kind == "powerlaw":
        rp, ci = pattern_powerlaw(rng, M, K, density)
    elif kind == "band":
        rp, ci = pattern_band_plus_uniform(rng, M, K, min(K, 16), density)
    else:
        raise ValueError(kind)
    return _finish(f"small_{kind}", rng, M, K, rp, ci, unit_values, Kd, N)


# ----------------------------------------------------------------------------------
# accounting helpers (sizes only)
# ----------------------------------------------------------------------------------

def flops(op: str, nnz: int, Kd: int, N: int) -> int:
    """2*nnz*width per stage; FusedMM is the sum of its two stages."""
    if op == "spmm":
        return 2 * nnz * N
    if op == "sddmm":
        return 2 * nnz * Kd
    if op == "fusedmm":
        return 2 * nnz * Kd + 2 * nnz * N
    raise ValueError(op)


def compulsory_bytes(op: str, M: int, K: int, nnz: int, Kd: int, N: int,
                     has_values: bool = True) -> int:
    """Bytes if every array is touched exactly once (row_ptr, col_idx, values, dense
    operands, output)."""
    R = 4 * (M + 1)
    I = 4 * nnz
    V = 4 * nnz if has_values else 0
    if op == "spmm":
        return R + I + V + 4 * K * N + 4 * M * N
    if op == "sddmm":
        return R + I + V + 4 * M * Kd + 4 * K * Kd + 4 * nnz
    if op == "fusedmm":
        return R + I + V + 4 * M * Kd + 4 * K * Kd + 4 * K * N + 4 * M * N
    raise ValueError(op)
