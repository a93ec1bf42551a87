"""Parity of the CUDA library (called through its C ABI) against the CPU oracle.

Floating-point gate, elementwise: |gpu - ref| <= 1e-5 * T + 1e-6, T = sum of |terms| of the
expanded sum that defines the element (returned by the oracle).  Integer side: the CSR pattern
arrays must be byte-identical after every call; hand-worked integer examples must match exactly.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2311_00368_b200 import workloads as W
from tests.util import read_golden

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-5, 1e-6


@pytest.fixture(scope="module")
def b():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2311_00368_b200 import binding
    return binding


def dev(x):
    return None if x is None else torch.from_numpy(np.ascontiguousarray(x)).cuda()


class DevProblem:
    def __init__(self, p, unit_as_null=False):
        self.p = p
        self.row_ptr, self.col_idx = dev(p.row_ptr), dev(p.col_idx)
        self.values = dev(p.values)
        self.A, self.B, self.D = dev(p.A), dev(p.B), dev(p.D)
        self._rp0, self._ci0 = self.row_ptr.clone(), self.col_idx.clone()

    def pattern_untouched(self):
        return torch.equal(self.row_ptr, self._rp0) and torch.equal(self.col_idx, self._ci0)


def gate(x, ref, T, what):
    x = x.detach().cpu().numpy().astype(np.float64)
    ok, ratio = oracle.within_tolerance(x, ref, T, RTOL, ATOL)
    assert ok, f"{what}: worst err/bound = {ratio:.3g}"
    return ratio


def check_all_ops(b, p, algos, null_values=False, ops=("spmm", "sddmm", "fusedmm")):
    d = DevProblem(p)
    sv_np = None if null_values else p.values
    sv = None if null_values else d.values
    for algo in algos:
        if "spmm" in ops and p.D is not None:
            ref, T = oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D)
            out = torch.full((p.M, p.N), float("nan"), device="cuda")
            b.spmm(d.row_ptr, d.col_idx, d.values, d.D, K=p.K, out=out, algo=algo)
            gate(out, ref, T, f"spmm algo={algo} {p.name}")
        if "sddmm" in ops and p.A is not None:
            ref, T = oracle.sddmm(p.row_ptr, p.col_idx, sv_np, p.A, p.B)
            out = torch.full((p.nnz,), float("nan"), device="cuda")
            b.sddmm(d.row_ptr, d.col_idx, sv, d.A, d.B, out=out, algo=algo)
            gate(out, ref, T, f"sddmm algo={algo} {p.name}")
        if "fusedmm" in ops and p.A is not None and p.D is not None:
            ref, T = oracle.fusedmm(p.row_ptr, p.col_idx, sv_np, p.A, p.B, p.D)
            out = torch.full((p.M, p.N), float("nan"), device="cuda")
            b.fusedmm(d.row_ptr, d.col_idx, sv, d.A, d.B, d.D, out=out, algo=algo)
            gate(out, ref, T, f"fusedmm algo={algo} {p.name}")
    torch.cuda.synchronize()
    assert d.pattern_untouched()


ROW_ALGOS = (1, 2)


def test_tiny_config(b):
    check_all_ops(b, W.tiny(), (0,) + ROW_ALGOS)
    check_all_ops(b, W.tiny(), ROW_ALGOS, null_values=True, ops=("sddmm", "fusedmm"))


def test_hand_worked_integer_example_exact(b):
    g, w = read_golden("fig1_csr.txt"), read_golden("fig1_worked.txt")
    for rows in (5, 4):
        ia = g["ia"].astype(np.int32)[: rows + 1]
        n = int(ia[-1])
        ja, av = g["ja"].astype(np.int32)[:n], g["avalue"].astype(np.float32)[:n]
        D = w["D"].astype(np.float32).reshape(4, 2)
        A = np.array([[i + 1, 1] for i in range(rows)], dtype=np.float32)
        B = np.array([[1, j] for j in range(4)], dtype=np.float32)
        for algo in ROW_ALGOS:
            O = b.spmm(dev(ia), dev(ja), dev(av), dev(D), algo=algo).cpu().numpy()
            assert np.array_equal(O, w["spmm"].reshape(5, 2)[:rows])
            C = b.sddmm(dev(ia), dev(ja), None, dev(A), dev(B), algo=algo).cpu().numpy()
            assert np.array_equal(C, w["sddmm_unit"][:n])
            C = b.sddmm(dev(ia), dev(ja), dev(av), dev(A), dev(B), algo=algo).cpu().numpy()
            assert np.array_equal(C, w["sddmm_scaled"][:n])
            E = b.fusedmm(dev(ia), dev(ja), dev(av), dev(A), dev(B), dev(D), algo=algo).cpu().numpy()
            assert np.array_equal(E, w["fused_scaled"].reshape(5, 2)[:rows])


@pytest.mark.parametrize("M,K,density,Kd,N,kind", [
    (300, 200, 0.2, 64, 64, "uniform"),      # SPLIT=2 geometry, KU=2
    (257, 333, 0.3, 128, 128, "uniform"),    # one float4 per lane, KU=4
    (129, 500, 0.25, 256, 256, "uniform"),   # two float4 per lane, KU=8
    (65, 700, 0.3, 260, 512, "uniform"),     # four float4 per lane, A row in shared memory
    (40, 300, 0.3, 32, 32, "uniform"),       # SPLIT=4 geometry
    (50, 256, 0.2, 100, 100, "uniform"),     # widths that are multiples of 4 but not of the slab
    (33, 260, 0.3, 132, 644, "uniform"),     # N > 512: two column slabs, ragged second slab
    (200, 256, 0.2, 128, 256, "powerlaw"),   # skewed rows incl. saturated rows
    (128, 256, 0.2, 64, 64, "band"),
    (31, 97, 0.3, 7, 5, "uniform"),          # odd widths: scalar kernels
    (64, 128, 0.3, 130, 130, "uniform"),     # widths = 2 mod 4: scalar kernels
    (1, 64, 0.5, 16, 16, "uniform"),         # single row
])
def test_small_shapes(b, M, K, density, Kd, N, kind):
    p = W.small_random(1000 + M, M, K, density, Kd, N, kind=kind)
    check_all_ops(b, p, ROW_ALGOS)
    check_all_ops(b, p, (1,), null_values=True, ops=("sddmm", "fusedmm"))


def _custom_rows(lens, K, seed, Kd=64, N=128):
    rng = np.random.default_rng(seed)
    cols = [np.sort(rng.choice(K, size=l, replace=False)).astype(np.int32) for l in lens]
    row_ptr = np.zeros(len(lens) + 1, dtype=np.int32)
    row_ptr[1:] = np.cumsum(lens)
    ci = np.concatenate(cols) if sum(lens) else np.zeros(0, np.int32)
    nnz = int(row_ptr[-1])
    return W.Problem("custom", len(lens), K, row_ptr, ci, W.values_uniform(rng, nnz), Kd, N,
                     W.dense_normal(rng, len(lens), Kd), W.dense_normal(rng, K, Kd),
                     W.dense_normal(rng, K, N))


def test_row_length_edges(b):
    """Empty rows, lengths around the 32-entry chunk and the 4-warp stride, one very long row."""
    lens = [0, 1, 31, 32, 33, 0, 127, 128, 129, 255, 256, 257, 4096, 0, 2, 64]
    check_all_ops(b, _custom_rows(lens, 4096, 5), ROW_ALGOS)


def test_all_rows_empty_and_zero_sizes(b):
    p = _custom_rows([0, 0, 0], 16, 6, Kd=8, N=8)
    d = DevProblem(p)
    out = torch.full((3, 8), float("nan"), device="cuda")
    b.spmm(d.row_ptr, d.col_idx, d.values, d.D, K=16, out=out)
    assert torch.equal(out, torch.zeros_like(out))
    out.fill_(float("nan"))
    b.fusedmm(d.row_ptr, d.col_idx, None, d.A, d.B, d.D, out=out)
    assert torch.equal(out, torch.zeros_like(out))
    assert b.sddmm(d.row_ptr, d.col_idx, None, d.A, d.B).numel() == 0
    # M = 0
    rp0 = torch.zeros(1, dtype=torch.int32, device="cuda")
    e_i = torch.zeros(0, dtype=torch.int32, device="cuda")
    e_f = torch.zeros(0, dtype=torch.float32, device="cuda")
    assert b.spmm(rp0, e_i, e_f, d.D, K=16).shape == (0, 8)


def test_unsorted_and_duplicate_entries(b):
    p = W.small_random(77, 90, 150, 0.3, 64, 128)
    rng = np.random.default_rng(3)
    ci, v = p.col_idx.copy(), p.values.copy()
    for i in range(p.M):
        a, e = p.row_ptr[i], p.row_ptr[i + 1]
        perm = a + rng.permutation(e - a)
        ci[a:e], v[a:e] = ci[perm], v[perm]
        if e - a >= 2:
            ci[a + 1] = ci[a]  # a duplicate column
    q = W.Problem("unsorted", p.M, p.K, p.row_ptr, ci, v, p.Kd, p.N, p.A, p.B, p.D)
    check_all_ops(b, q, ROW_ALGOS)


def test_leading_dimensions_and_inplace_sddmm(b):
    p = W.small_random(55, 70, 120, 0.3, 64, 128)
    d = DevProblem(p)
    pad = lambda t, extra: torch.cat([t, torch.full((t.shape[0], extra), 7.0, device="cuda")], 1)[:, : t.shape[1]]
    A, B, D = pad(d.A, 4), pad(d.B, 8), pad(d.D, 12)
    assert A.stride(0) == 68 and D.stride(0) == 140
    obuf = torch.full((p.M, p.N + 4), -3.0, device="cuda")
    out = obuf[:, : p.N]
    ref, T = oracle.fusedmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D)
    b.fusedmm(d.row_ptr, d.col_idx, d.values, A, B, D, out=out)
    gate(out, ref, T, "fusedmm ld")
    assert torch.all(obuf[:, p.N:] == -3.0)  # padding columns of O untouched
    ref, T = oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D)
    b.spmm(d.row_ptr, d.col_idx, d.values, D, out=out)
    gate(out, ref, T, "spmm ld")
    # odd leading dimension -> scalar path
    D3 = pad(d.D, 3)
    b.spmm(d.row_ptr, d.col_idx, d.values, D3, out=out)
    gate(out, ref, T, "spmm odd ld")
    # in-place SDDMM: out_values aliases s_values
    ref, T = oracle.sddmm(p.row_ptr, p.col_idx, p.values, p.A, p.B)
    vals = d.values.clone()
    b.sddmm(d.row_ptr, d.col_idx, vals, A, B, out=vals)
    gate(vals, ref, T, "sddmm in place")


def test_argument_errors(b):
    p = W.small_random(9, 8, 8, 0.5, 8, 8)
    d = DevProblem(p)
    with pytest.raises(b.B2spError) as e:
        b.spmm(d.row_ptr, d.col_idx, d.values, d.D, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 5
    with pytest.raises(b.B2spError) as e:
        b.spmm(d.row_ptr, d.col_idx, d.values, d.D, algo=9)
    assert e.value.status == 1
    st = b.lib.b2sp_spmm(8, 8, 8, -1, None, None, None, None, 8, None, 8, None, 0, 0, None)
    assert st == 1
    assert b.validate_csr(d.row_ptr, d.col_idx, 8)
    bad = d.col_idx.clone()
    bad[0] = 8
    assert not b.validate_csr(d.row_ptr, bad, 8)
    rp = d.row_ptr.clone()
    rp[2] = rp[1] - 1 if int(rp[1]) > 0 else 5
    assert not b.validate_csr(rp, d.col_idx, 8)


def test_host_buffer_entry_points(b):
    p = W.small_random(19, 100, 90, 0.2, 64, 64)
    t = lambda x: torch.from_numpy(x).pin_memory()
    rp, ci, v, A, B, D = t(p.row_ptr), t(p.col_idx), t(p.values), t(p.A), t(p.B), t(p.D)
    O = torch.empty((p.M, p.N), dtype=torch.float32).pin_memory()
    ref, T = oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D)
    gate(b.spmm_host(rp, ci, v, D, O), ref, T, "spmm_host")
    ref, T = oracle.fusedmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D)
    gate(b.fusedmm_host(rp, ci, v, A, B, D, O), ref, T, "fusedmm_host")
    C = torch.empty(p.nnz, dtype=torch.float32).pin_memory()
    ref, T = oracle.sddmm(p.row_ptr, p.col_idx, None, p.A, p.B)
    gate(b.sddmm_host(rp, ci, None, A, B, C), ref, T, "sddmm_host")


# ---- the named full-size workloads -------------------------------------------------------------

def test_config_spmm_full(b):
    p = W.spmm_case()
    d = DevProblem(p)
    ref, T = oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D)
    for algo in (0, 1, 2):
        gate(b.spmm(d.row_ptr, d.col_idx, d.values, d.D, algo=algo), ref, T, "spmm config")


def test_config_sddmm_full(b):
    p = W.sddmm_case()
    d = DevProblem(p)
    ref, T = oracle.sddmm(p.row_ptr, p.col_idx, p.values, p.A, p.B)
    for algo in (0, 1):
        gate(b.sddmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, algo=algo), ref, T, "sddmm config")
    gate(b.sddmm(d.row_ptr, d.col_idx, None, d.A, d.B), ref, T, "sddmm config, NULL values")


def test_config_attention_fused_equals_separate_launches(b):
    for prob in (0, 7):   # (every element of all eight problems: tests/test_gpu_configs.py)
        p = W.attention_case(prob)
        # fused == separate launches on the GPU too (C rounded to fp32 in between)
        d = DevProblem(p)
        C = b.sddmm(d.row_ptr, d.col_idx, d.values, d.A, d.B)
        O2 = b.spmm(d.row_ptr, d.col_idx, C, d.D)
        O1 = b.fusedmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, d.D)
        scale = float(O1.abs().max())
        assert float((O1 - O2).abs().max()) <= 1e-4 * scale


def test_device_status_is_reset_by_every_family(b):
    """b2sp_device_status reports the last call on a workspace: a stale word (here: garbage left in the
    buffer) must not survive a call of any kernel family."""
    p = W.small_random(77, 300, 400, 0.2, 32, 64)
    d = DevProblem(p)
    n = max(b.workspace_bytes(op, p.M, p.K, p.Kd, p.N, p.nnz) for op in range(3))
    for algo in (0, 1, 2, 3):
        ws = torch.full((max(n, 1 << 20),), 0x5a, dtype=torch.uint8, device="cuda")
        assert b.device_status(ws) != 0
        b.spmm(d.row_ptr, d.col_idx, d.values, d.D, workspace=ws, algo=algo)
        assert b.device_status(ws) == 0, f"spmm algo={algo}"
        ws.fill_(0x5a)
        b.sddmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, workspace=ws, algo=algo)
        assert b.device_status(ws) == 0, f"sddmm algo={algo}"
        ws.fill_(0x5a)
        b.fusedmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, d.D, workspace=ws, algo=algo)
        assert b.device_status(ws) == 0, f"fusedmm algo={algo}"
