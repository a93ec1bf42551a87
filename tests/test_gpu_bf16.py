"""The three ops with bfloat16 dense operands and fp32 accumulation (b2sp_*_bf16), against the CPU oracle.

Reading of the tolerance: the inputs of the problem ARE the bfloat16 values.  The fp32 operands a generator
draws are rounded to bfloat16 on the host, the unchanged fp64 oracle runs on the rounded values, and the
gate is the one of the fp32 ops, |gpu - ref| <= 1e-5 * T + 1e-6 with T the sum of |terms| -- products of two
bfloat16 numbers are exact in fp32, so only the fp32 summation order separates the GPU result from the
exact one.  The stored values of S stay fp32.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2311_00368_b200 import workloads as W
from tests.test_gpu_parity import gate

pytestmark = pytest.mark.gpu

ROW, ROW_NAT, TILE, PREPARED = 1, 2, 3, 4
BF = torch.bfloat16


@pytest.fixture(scope="module")
def b():
    assert torch.cuda.is_available()
    from paper_2311_00368_b200 import binding
    return binding


def round_bf16(x):
    """fp32 array -> (the same values rounded to bfloat16, as fp32 numpy; the bfloat16 CUDA tensor)."""
    t = torch.from_numpy(np.ascontiguousarray(x)).to(BF)
    return t.to(torch.float32).numpy(), t.cuda()


class Bf16Problem:
    def __init__(self, p):
        self.p = p
        dev = lambda x: torch.from_numpy(np.ascontiguousarray(x)).cuda()
        self.row_ptr, self.col_idx, self.values = dev(p.row_ptr), dev(p.col_idx), dev(p.values)
        self.A32 = self.B32 = self.D32 = self.A = self.B = self.D = None
        if p.A is not None:
            self.A32, self.A = round_bf16(p.A)
            self.B32, self.B = round_bf16(p.B)
        if p.D is not None:
            self.D32, self.D = round_bf16(p.D)
        self._rp0, self._ci0 = self.row_ptr.clone(), self.col_idx.clone()

    def refs(self, ops, null_values=False):
        p, sv = self.p, None if null_values else self.p.values
        r = {}
        if "spmm" in ops:
            r["spmm"] = oracle.spmm(p.row_ptr, p.col_idx, p.values, self.D32)
        if "sddmm" in ops:
            r["sddmm"] = oracle.sddmm(p.row_ptr, p.col_idx, sv, self.A32, self.B32)
        if "fusedmm" in ops:
            r["fusedmm"] = oracle.fusedmm(p.row_ptr, p.col_idx, sv, self.A32, self.B32, self.D32)
        return r


def run(b, d, refs, algo, ws, expect, null_values=False, tag=""):
    p = d.p
    sv = None if null_values else d.values
    worst = 0.0
    for op, (ref, T) in refs.items():
        if op == "spmm":
            out = torch.full((p.M, p.N), float("nan"), device="cuda")
            b.spmm(d.row_ptr, d.col_idx, d.values, d.D, K=p.K, out=out, workspace=ws, algo=algo, dtype=BF)
            idx = b.OP_SPMM
        elif op == "sddmm":
            out = torch.full((p.nnz,), float("nan"), device="cuda")
            b.sddmm(d.row_ptr, d.col_idx, sv, d.A, d.B, out=out, workspace=ws, algo=algo, dtype=BF)
            idx = b.OP_SDDMM
        else:
            out = torch.full((p.M, p.N), float("nan"), device="cuda")
            b.fusedmm(d.row_ptr, d.col_idx, sv, d.A, d.B, d.D, out=out, workspace=ws, algo=algo, dtype=BF)
            idx = b.OP_FUSEDMM
        if expect is not None:
            assert b.last_algo(idx) in expect, f"{op} bf16 algo={algo}: ran family {b.last_algo(idx)}"
        assert b.device_status(ws) == 0
        worst = max(worst, gate(out, ref, T, f"{op} bf16 algo={algo} {p.name} {tag}"))
    assert torch.equal(d.row_ptr, d._rp0) and torch.equal(d.col_idx, d._ci0)
    return worst


def every_family(b, p, ops=("spmm", "sddmm", "fusedmm"), tile=True):
    d = Bf16Problem(p)
    refs = d.refs(ops)
    ws = torch.empty(max(max(b.workspace_bytes(i, p.M, p.K, p.Kd, p.N, p.nnz) for i in range(3)), 1 << 20),
                     dtype=torch.uint8, device="cuda")
    run(b, d, refs, ROW, ws, (ROW,))
    run(b, d, refs, ROW_NAT, ws, (ROW_NAT,))
    if tile:
        run(b, d, refs, TILE, ws, (TILE,))
        b.prepare_pattern(d.row_ptr, d.col_idx, p.K, ws)
        run(b, d, refs, PREPARED, ws, (TILE,), tag="prepared")
        run(b, d, refs, PREPARED, ws, (TILE,), tag="prepared, again")
    return d, ws


@pytest.mark.parametrize("M,K,density,Kd,N,kind", [
    (256, 256, 0.10, 64, 64, "uniform"),      # the tiny configuration's shape
    (257, 333, 0.30, 128, 128, "uniform"),    # ragged M and K
    (300, 512, 0.20, 100, 100, "uniform"),    # widths padded inside the tf32 copies
    (130, 1024, 0.25, 24, 300, "uniform"),    # three O column tiles; N > 256 takes the two-phase path on tiles
    (512, 2048, 0.10, 128, 256, "uniform"),   # several K splits
    (384, 1024, 0.20, 64, 128, "powerlaw"),   # skewed rows incl. full rows
    (256, 512, 0.20, 32, 32, "band"),
    (260, 700, 0.20, 48, 63, "uniform"),      # odd width: scalar row kernels, plain stores in the tile flush
    (65, 700, 0.30, 260, 512, "uniform"),     # Kd > 128: row kernels only (A row in shared memory)
])
def test_bf16_shapes_every_family(b, M, K, density, Kd, N, kind):
    p = W.small_random(6000 + M + N, M, K, density, Kd, N, kind=kind)
    d, ws = every_family(b, p, tile=Kd <= 128)
    # all-ones sampling pattern
    run(b, d, d.refs(("sddmm", "fusedmm"), null_values=True), TILE if Kd <= 128 else ROW, ws, None, null_values=True)


def test_bf16_exact_on_small_integers(b):
    """Small integers are exact in bfloat16 and every partial sum is exact in fp32: bit-equal results."""
    rng = np.random.default_rng(8)
    p = W.small_random(6100, 256, 256, 0.3, 32, 64)
    p.values[:] = rng.integers(-2, 3, p.nnz).astype(np.float32)
    p.A[:] = rng.integers(-3, 4, p.A.shape).astype(np.float32)
    p.B[:] = rng.integers(-3, 4, p.B.shape).astype(np.float32)
    p.D[:] = rng.integers(-4, 5, p.D.shape).astype(np.float32)
    d = Bf16Problem(p)
    refs = d.refs(("spmm", "sddmm", "fusedmm"))
    ws = torch.empty(64 << 20, dtype=torch.uint8, device="cuda")
    for algo in (ROW, TILE):
        O = b.fusedmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, d.D, workspace=ws, algo=algo, dtype=BF)
        assert np.array_equal(O.cpu().numpy().astype(np.float64), refs["fusedmm"][0])
        C = b.sddmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, workspace=ws, algo=algo, dtype=BF)
        assert np.array_equal(C.cpu().numpy().astype(np.float64), refs["sddmm"][0])
        O = b.spmm(d.row_ptr, d.col_idx, d.values, d.D, workspace=ws, algo=algo, dtype=BF)
        assert np.array_equal(O.cpu().numpy().astype(np.float64), refs["spmm"][0])


def test_bf16_leading_dimensions_unsorted_rows_and_dtype_check(b):
    p = W.small_random(6200, 200, 300, 0.3, 64, 128)
    rng = np.random.default_rng(3)
    ci, v = p.col_idx.copy(), p.values.copy()
    a, e = p.row_ptr[7], p.row_ptr[8]
    perm = a + rng.permutation(e - a)
    ci[a:e], v[a:e] = ci[perm], v[perm]
    q = W.Problem("unsorted", p.M, p.K, p.row_ptr, ci, v, p.Kd, p.N, p.A, p.B, p.D)
    d = Bf16Problem(q)
    refs = d.refs(("spmm", "sddmm", "fusedmm"))
    ws = torch.empty(64 << 20, dtype=torch.uint8, device="cuda")
    run(b, d, refs, TILE, ws, (TILE,), tag="unsorted row: fallback to the bf16 row kernels")
    # padded leading dimensions (multiples of 8 and not)
    for pad in (8, 4, 3):
        widen = lambda t: torch.cat([t, torch.full((t.shape[0], pad), 7.0, device="cuda", dtype=BF)], 1)[:, :t.shape[1]]
        d2 = Bf16Problem(q)
        d2.A, d2.B, d2.D = widen(d.A), widen(d.B), widen(d.D)
        assert d2.D.stride(0) == q.N + pad
        for algo in (ROW, TILE):
            run(b, d2, refs, algo, ws, None, tag=f"ld padded by {pad}")
    with pytest.raises(TypeError):
        b.spmm(d.row_ptr, d.col_idx, d.values, d.D.float(), workspace=ws, dtype=BF)


def test_bf16_configs_every_element(b):
    """SPMM and SDDMM configurations, one attention problem and the bench workload, bfloat16 operands."""
    every_family(b, W.spmm_case(), ops=("spmm",))
    every_family(b, W.sddmm_case(), ops=("sddmm",))
    every_family(b, W.attention_case(2))
    d, ws = every_family(b, W.sweep_case(0.3, 128))
    w = run(b, d, d.refs(("spmm", "sddmm", "fusedmm")), 0, ws, (TILE,), tag="auto")
    assert w < 0.5


def test_bf16_non_finite_values_in_unreferenced_rows(b):
    """As for fp32 operands: an Inf or NaN in a row of B or D that no stored entry names must not reach the
    outputs; the operand pre-pass sees it and the bf16 row kernels produce the call's result."""
    p = W.small_random(6300, 300, 700, 0.2, 64, 128)
    dead = np.array([5, 77])
    keep = ~np.isin(p.col_idx, dead)
    lens = np.add.reduceat(keep.astype(np.int64), p.row_ptr[:-1].astype(np.int64))
    rp = np.zeros(p.M + 1, dtype=np.int32)
    rp[1:] = np.cumsum(lens)
    q = W.Problem("holes", p.M, p.K, rp, p.col_idx[keep], p.values[keep], p.Kd, p.N, p.A, p.B.copy(), p.D.copy())
    d = Bf16Problem(q)
    refs = d.refs(("spmm", "sddmm", "fusedmm"))        # from the clean operands
    d.D[5, :] = float("nan")
    d.B[77, :] = float("inf")
    ws = torch.empty(64 << 20, dtype=torch.uint8, device="cuda")
    run(b, d, refs, TILE, ws, (TILE,), tag="NaN / Inf in unreferenced rows")
    flags = ws[320:332].view(torch.int32).cpu().numpy()
    assert flags[1] == 0 and flags[2] == 0
