"""The seeded generators: CSR validity, densities, band/power-law structure, determinism."""
import numpy as np
import pytest

from paper_2311_00368_b200 import workloads as W


def _check_csr(p):
    assert p.row_ptr.dtype == np.int32 and p.col_idx.dtype == np.int32 and p.values.dtype == np.float32
    assert p.row_ptr[0] == 0 and len(p.row_ptr) == p.M + 1
    lens = np.diff(p.row_ptr)
    assert lens.min() >= 0 and p.row_ptr[-1] == len(p.col_idx) == len(p.values)
    assert p.col_idx.min() >= 0 and p.col_idx.max() < p.K
    # sorted and unique inside each row
    d = np.diff(p.col_idx.astype(np.int64))
    row_start = np.zeros(p.nnz, dtype=bool)
    row_start[p.row_ptr[:-1][lens > 0]] = True
    assert np.all(d[~row_start[1:]] > 0)


def test_tiny_is_deterministic_and_valid():
    a, b = W.tiny(), W.tiny()
    _check_csr(a)
    assert np.array_equal(a.col_idx, b.col_idx) and np.array_equal(a.D, b.D)
    assert a.A.shape == (256, 64) and a.B.shape == (256, 64) and a.D.shape == (256, 64)
    assert abs(a.nnz / 256 ** 2 - 0.10) < 0.01
    assert np.all(np.abs(a.values) <= 1.0) and a.values.std() > 0.4


def test_band_plus_uniform_structure():
    p = W.attention_case(0, L=1024, head_dim=16)
    _check_csr(p)
    assert abs(p.nnz / 1024 ** 2 - 0.20) < 0.01
    assert np.all(p.values == 1.0)
    rows = np.repeat(np.arange(p.M), np.diff(p.row_ptr))
    present = set(zip(rows.tolist(), p.col_idx.tolist()))
    for i in (0, 1, 63, 64, 300, 1023):
        for j in range(max(0, i - 64), min(1024, i + 64)):
            assert (i, j) in present
    assert W.band_entry_count(4096, 4096, 64) == 520192
    q = W.attention_case(1, L=1024, head_dim=16)
    assert not np.array_equal(p.col_idx[:1000], q.col_idx[:1000])


@pytest.mark.parametrize("density", [0.1, 0.3])
def test_powerlaw_lengths(density):
    M = K = 1024
    lens = W.powerlaw_row_lengths(M, K, density)
    assert lens.sum() == round(density * M * K)
    assert np.all(np.diff(lens) <= 0) and lens.max() <= K and lens.min() >= 1
    p = W.small_random(4, 256, 256, density, 8, 8, kind="powerlaw")
    _check_csr(p)
    assert p.nnz == round(density * 256 * 256)
    got = np.sort(np.diff(p.row_ptr))[::-1]
    assert np.array_equal(got, W.powerlaw_row_lengths(256, 256, density))


def test_powerlaw_full_size_statistics():
    """Shape of the 8192^2 sweep pattern (lengths only; no columns drawn)."""
    for density, saturated in ((0.1, 199), (0.2, 470), (0.3, 799)):
        lens = W.powerlaw_row_lengths(8192, 8192, density)
        assert abs(int((lens == 8192).sum()) - saturated) <= 2
        top = np.sort(lens)[::-1][:819].sum() / lens.sum()
        assert 0.3 < top < 0.6
