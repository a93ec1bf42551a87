"""Pins for the CPU oracle: each test checks it against something other than itself --
values the paper prints (Fig. 1), hand-worked integer examples, the dense definitions of
Eq. 1-3 evaluated by numpy on the densified pattern, closed forms and invariants."""
import numpy as np
import pytest

import oracle
from paper_2311_00368_b200 import workloads as W
from tests.util import csr_rows, csr_to_dense, dense_to_csr, read_golden


@pytest.fixture(scope="module")
def fig1():
    g = read_golden("fig1_csr.txt")
    w = read_golden("fig1_worked.txt")
    return g, w


def test_fig1_csr_convention(fig1):
    """Paper Fig. 1: the printed dense matrix and the printed ia/ja/avalue describe the same
    matrix under the 0-based, row-ordered convention the oracle reads."""
    g, _ = fig1
    rp, ci, v = dense_to_csr(g["dense"])
    assert rp.tolist() == g["ia"].astype(int).tolist()
    assert ci.tolist() == g["ja"].astype(int).tolist()
    assert v.tolist() == g["avalue"].tolist()
    # SPMM with D = identity must reproduce the dense matrix from the *printed* arrays.
    ia, ja = g["ia"].astype(np.int32), g["ja"].astype(np.int32)
    O, _ = oracle.spmm(ia, ja, g["avalue"].astype(np.float32), np.eye(4, dtype=np.float32))
    assert np.array_equal(O, g["dense"])


@pytest.mark.parametrize("rows", [5, 4])
def test_hand_worked_example(fig1, rows):
    """Integer example worked by hand on Fig. 1's matrix (5x4, and its first 4 rows as a 4x4)."""
    g, w = fig1
    ia = g["ia"].astype(np.int32)[: rows + 1]
    n = int(ia[-1])
    ja = g["ja"].astype(np.int32)[:n]
    av = g["avalue"].astype(np.float32)[:n]
    D = w["D"].astype(np.float32).reshape(4, 2)
    A = np.array([[i + 1, 1] for i in range(rows)], dtype=np.float32)
    B = np.array([[1, j] for j in range(4)], dtype=np.float32)
    O, T = oracle.spmm(ia, ja, av, D)
    assert np.array_equal(O, w["spmm"].reshape(5, 2)[:rows])
    assert np.array_equal(T, O)  # all terms positive => sum|terms| == sum
    C, _ = oracle.sddmm(ia, ja, None, A, B)
    assert np.array_equal(C, w["sddmm_unit"][:n])
    C, _ = oracle.sddmm(ia, ja, av, A, B)
    assert np.array_equal(C, w["sddmm_scaled"][:n])
    E, _ = oracle.fusedmm(ia, ja, av, A, B, D)
    assert np.array_equal(E, w["fused_scaled"].reshape(5, 2)[:rows])


def _adversarial(M, K, seed):
    """Random pattern with an empty row, a full row and a single-entry row."""
    rng = np.random.default_rng(seed)
    mask = rng.random((M, K)) < 0.3
    mask[0] = False
    if M > 1:
        mask[1] = True
    if M > 2:
        mask[2] = False
        mask[2, K - 1] = True
    dense = np.where(mask, rng.uniform(-1, 1, (M, K)), 0.0).astype(np.float32)
    return dense


@pytest.mark.parametrize("M,K,Kd,N,seed", [(7, 5, 3, 4, 0), (33, 64, 17, 9, 1), (64, 40, 32, 64, 2),
                                           (1, 1, 1, 1, 3), (12, 50, 5, 130, 4)])
def test_against_dense_definitions(M, K, Kd, N, seed):
    """Eq. 1-3 on the densified matrix, via numpy matmul in fp64 (a different code path:
    no CSR traversal)."""
    dense = _adversarial(M, K, seed)
    rp, ci, v = dense_to_csr(dense)
    rng = np.random.default_rng(100 + seed)
    A = rng.standard_normal((M, Kd)).astype(np.float32)
    B = rng.standard_normal((K, Kd)).astype(np.float32)
    D = rng.standard_normal((K, N)).astype(np.float32)
    S64 = dense.astype(np.float64)
    rows = csr_rows(rp)

    O, T = oracle.spmm(rp, ci, v, D)
    np.testing.assert_allclose(O, S64 @ D.astype(np.float64), rtol=0, atol=1e-12)
    np.testing.assert_allclose(T, np.abs(S64) @ np.abs(D.astype(np.float64)), rtol=0, atol=1e-12)

    P = A.astype(np.float64) @ B.astype(np.float64).T
    C, TC = oracle.sddmm(rp, ci, v, A, B)
    np.testing.assert_allclose(C, (P * S64)[rows, ci], rtol=0, atol=1e-12)
    Pabs = np.abs(A.astype(np.float64)) @ np.abs(B.astype(np.float64)).T
    np.testing.assert_allclose(TC, (Pabs * np.abs(S64))[rows, ci], rtol=0, atol=1e-12)
    C1, _ = oracle.sddmm(rp, ci, None, A, B)
    np.testing.assert_allclose(C1, P[rows, ci], rtol=0, atol=1e-12)

    E, TE = oracle.fusedmm(rp, ci, v, A, B, D)
    np.testing.assert_allclose(E, (P * S64) @ D.astype(np.float64), rtol=0, atol=1e-11)
    np.testing.assert_allclose(TE, (Pabs * np.abs(S64)) @ np.abs(D.astype(np.float64)),
                               rtol=0, atol=1e-11)
    mask = (dense != 0).astype(np.float64)
    E1, _ = oracle.fusedmm(rp, ci, None, A, B, D)
    np.testing.assert_allclose(E1, (P * mask) @ D.astype(np.float64), rtol=0, atol=1e-11)


def test_duplicates_and_unsorted_entries():
    """Each stored entry is its own term / own output slot, whatever the order."""
    rp = np.array([0, 4, 4, 6], dtype=np.int32)
    ci = np.array([3, 0, 3, 1, 2, 2], dtype=np.int32)
    v = np.array([1.5, -2.0, 0.25, 4.0, 1.0, -1.0], dtype=np.float32)
    rng = np.random.default_rng(7)
    A = rng.standard_normal((3, 6)).astype(np.float32)
    B = rng.standard_normal((4, 6)).astype(np.float32)
    D = rng.standard_normal((4, 5)).astype(np.float32)
    S = csr_to_dense(3, 4, rp, ci, v)  # duplicates accumulate
    O, _ = oracle.spmm(rp, ci, v, D)
    np.testing.assert_allclose(O, S @ D.astype(np.float64), atol=1e-12)
    assert np.array_equal(O[1], np.zeros(5))  # empty row
    assert np.allclose(O[2], 0.0)  # +1 and -1 on the same column cancel
    P = A.astype(np.float64) @ B.astype(np.float64).T
    C, _ = oracle.sddmm(rp, ci, v, A, B)
    rows = csr_rows(rp)
    np.testing.assert_allclose(C, v.astype(np.float64) * P[rows, ci], atol=1e-12)


def test_fused_equals_spmm_of_sddmm():
    """Alg. 3 wiring: FusedMM == SPMM(SDDMM(.)) in fp64 (the intermediate is rounded to fp32
    only when it is passed back in, so compare with the unrounded product by hand)."""
    p = W.small_random(11, 96, 80, 0.2, 24, 40)
    C, _ = oracle.sddmm(p.row_ptr, p.col_idx, p.values, p.A, p.B)
    E, _ = oracle.fusedmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D)
    rows = csr_rows(p.row_ptr)
    ref = np.zeros((p.M, p.N))
    np.add.at(ref, rows, C[:, None] * p.D.astype(np.float64)[p.col_idx])
    np.testing.assert_allclose(E, ref, rtol=1e-12, atol=1e-12)
    # and through the oracle's own SPMM with C rounded to fp32: equal up to that rounding
    O, T = oracle.spmm(p.row_ptr, p.col_idx, C.astype(np.float32), p.D)
    assert np.all(np.abs(O - E) <= 1e-7 * T + 1e-12)


def test_closed_forms():
    p = W.small_random(5, 50, 70, 0.25, 16, 12)
    lens = np.diff(p.row_ptr).astype(np.float64)
    ones_D = np.ones((p.K, 3), dtype=np.float32)
    O, _ = oracle.spmm(p.row_ptr, p.col_idx, W.values_ones(p.nnz), ones_D)
    assert np.array_equal(O, np.repeat(lens[:, None], 3, axis=1))  # row length
    O, _ = oracle.spmm(p.row_ptr, p.col_idx, p.values, ones_D)
    rowsum = np.zeros(p.M)
    np.add.at(rowsum, csr_rows(p.row_ptr), p.values.astype(np.float64))
    np.testing.assert_allclose(O[:, 0], rowsum, atol=1e-12)
    # A = B = ones => C[p] = s_p * Kd
    onesA = np.ones((p.M, p.Kd), dtype=np.float32)
    onesB = np.ones((p.K, p.Kd), dtype=np.float32)
    C, T = oracle.sddmm(p.row_ptr, p.col_idx, p.values, onesA, onesB)
    assert np.array_equal(C, p.values.astype(np.float64) * p.Kd)
    assert np.array_equal(T, np.abs(p.values.astype(np.float64)) * p.Kd)
    # S = identity: SPMM returns D, SDDMM returns row-wise dots, fused scales D rows by them
    n = 9
    rp = np.arange(n + 1, dtype=np.int32)
    ci = np.arange(n, dtype=np.int32)
    rng = np.random.default_rng(1)
    A = rng.standard_normal((n, 4)).astype(np.float32)
    B = rng.standard_normal((n, 4)).astype(np.float32)
    D = rng.standard_normal((n, 6)).astype(np.float32)
    O, _ = oracle.spmm(rp, ci, np.ones(n, np.float32), D)
    assert np.array_equal(O, D.astype(np.float64))
    dots = (A.astype(np.float64) * B.astype(np.float64)).sum(axis=1)
    C, _ = oracle.sddmm(rp, ci, None, A, B)
    np.testing.assert_allclose(C, dots, atol=1e-13)
    E, _ = oracle.fusedmm(rp, ci, None, A, B, D)
    np.testing.assert_allclose(E, dots[:, None] * D, atol=1e-12)


def test_fully_dense_equals_textbook_gemm():
    """S with every entry stored: the ops are plain dense products (triple loop)."""
    M, K, Kd, N = 5, 6, 4, 3
    rng = np.random.default_rng(3)
    Sd = rng.uniform(-1, 1, (M, K)).astype(np.float32)
    rp = (np.arange(M + 1) * K).astype(np.int32)
    ci = np.tile(np.arange(K, dtype=np.int32), M)
    A = rng.standard_normal((M, Kd)).astype(np.float32)
    B = rng.standard_normal((K, Kd)).astype(np.float32)
    D = rng.standard_normal((K, N)).astype(np.float32)
    gemm = [[sum(float(Sd[i, k]) * float(D[k, n]) for k in range(K)) for n in range(N)] for i in range(M)]
    O, _ = oracle.spmm(rp, ci, Sd.reshape(-1), D)
    np.testing.assert_allclose(O, np.array(gemm), atol=1e-13)
    abt = [[sum(float(A[i, l]) * float(B[k, l]) for l in range(Kd)) for k in range(K)] for i in range(M)]
    C, _ = oracle.sddmm(rp, ci, None, A, B)
    np.testing.assert_allclose(C.reshape(M, K), np.array(abt), atol=1e-13)


def test_linearity_and_permutations():
    p = W.small_random(21, 40, 60, 0.3, 8, 10)
    rng = np.random.default_rng(2)
    D2 = rng.standard_normal(p.D.shape).astype(np.float32)
    O1, _ = oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D)
    O2, _ = oracle.spmm(p.row_ptr, p.col_idx, p.values, D2)
    # D + D2 rounded to fp32 would not be exactly linear; use exactly representable halves
    Dh = (p.D * np.float32(0.5)).astype(np.float32)
    Oh, _ = oracle.spmm(p.row_ptr, p.col_idx, p.values, Dh)
    np.testing.assert_allclose(Oh, 0.5 * O1, rtol=0, atol=0)
    S = csr_to_dense(p.M, p.K, p.row_ptr, p.col_idx, p.values)
    np.testing.assert_allclose(O1 + O2, S @ (p.D.astype(np.float64) + D2.astype(np.float64)), atol=1e-11)
    # permute the entries inside every row (columns and values together)
    ci, v = p.col_idx.copy(), p.values.copy()
    perm = np.arange(p.nnz)
    for i in range(p.M):
        a, b = p.row_ptr[i], p.row_ptr[i + 1]
        perm[a:b] = a + rng.permutation(b - a)
    ci, v = ci[perm], v[perm]
    Op, _ = oracle.spmm(p.row_ptr, ci, v, p.D)
    np.testing.assert_allclose(Op, O1, rtol=0, atol=1e-12)
    C, _ = oracle.sddmm(p.row_ptr, p.col_idx, p.values, p.A, p.B)
    Cp, _ = oracle.sddmm(p.row_ptr, ci, v, p.A, p.B)
    assert np.array_equal(Cp, C[perm])
    E, _ = oracle.fusedmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D)
    Ep, _ = oracle.fusedmm(p.row_ptr, ci, v, p.A, p.B, p.D)
    np.testing.assert_allclose(Ep, E, rtol=0, atol=1e-11)


def test_row_range_variants_match_full():
    p = W.small_random(31, 64, 48, 0.2, 12, 20)
    O, T = oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D)
    Or, Tr = oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D, rows=(10, 33))
    assert np.array_equal(Or, O[10:33]) and np.array_equal(Tr, T[10:33])
    C, _ = oracle.sddmm(p.row_ptr, p.col_idx, p.values, p.A, p.B)
    Cr, _ = oracle.sddmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, rows=(10, 33))
    assert np.array_equal(Cr, C[p.row_ptr[10]:p.row_ptr[33]])
    E, _ = oracle.fusedmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D)
    Er, _ = oracle.fusedmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D, rows=(10, 33))
    assert np.array_equal(Er, E[10:33])


def test_result_independent_of_thread_count(monkeypatch):
    """Rows are independent: rerunning gives bit-identical results (dynamic schedule)."""
    p = W.small_random(41, 200, 100, 0.2, 16, 16)
    E1, _ = oracle.fusedmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D)
    E2, _ = oracle.fusedmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D)
    assert np.array_equal(E1, E2)


def test_byte_and_flop_accounting_matches_paper():
    """Performance Analysis section: worst-case arithmetic intensity 0.49 at N=128 (every
    gathered dense row re-read: 2N flop per 4N+8 bytes) and ~57 when each array is loaded once
    (M=K=8192, N=128, 30% density; loads only)."""
    N = 128
    assert abs(2 * N / (4 * N + 8) - 0.49) < 0.005
    M = K = 8192
    nnz = int(0.3 * M * K)
    fl = W.flops("sddmm", nnz, N, 0)
    loads = W.compulsory_bytes("sddmm", M, K, nnz, N, 0, has_values=False) - 4 * nnz
    assert abs(fl / loads - 57) < 1.5
    assert W.flops("fusedmm", nnz, 128, 64) == W.flops("sddmm", nnz, 128, 0) + W.flops("spmm", nnz, 0, 64)
    assert (W.compulsory_bytes("sddmm", M, K, nnz, 128, 0) + W.compulsory_bytes("spmm", M, K, nnz, 0, 64)
            - W.compulsory_bytes("fusedmm", M, K, nnz, 128, 64)) == 12 * nnz + 4 * (M + 1)


def test_tolerance_gate():
    ok, r = oracle.within_tolerance(np.array([1.0 + 5e-6]), np.array([1.0]), np.array([1.0]))
    assert ok and 0.4 < r < 0.5
    ok, _ = oracle.within_tolerance(np.array([1.0 + 2e-5]), np.array([1.0]), np.array([1.0]))
    assert not ok
    ok, _ = oracle.within_tolerance(np.array([np.nan]), np.array([1.0]), np.array([1.0]))
    assert not ok
