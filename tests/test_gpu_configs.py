"""Full-size parity: every element of every output of the five named configurations (and of a few
cases of the paper's evaluation grid), for every kernel family that accepts the sizes, against the
CPU oracle.  Gate as everywhere: |gpu - ref| <= 1e-5 * T + 1e-6 elementwise, T = sum of |terms|;
the CSR pattern arrays must be byte-identical after the calls.

The families: the CUDA-core row kernels (binned order), the dense-tile kernels called statelessly, and
the dense-tile kernels on ONE window table prepared once and shared by the three ops -- the launch
configuration bench.py times.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2311_00368_b200 import workloads as W
from tests.test_gpu_parity import DevProblem, gate

pytestmark = pytest.mark.gpu

ROW, TILE, PREPARED = 1, 3, 4
OPS = ("spmm", "sddmm", "fusedmm")


@pytest.fixture(scope="module")
def b():
    assert torch.cuda.is_available()
    from paper_2311_00368_b200 import binding
    return binding


def oracle_refs(p, ops, null_values=False):
    sv = None if null_values else p.values
    refs = {}
    if "spmm" in ops:
        refs["spmm"] = oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D)
    if "sddmm" in ops:
        refs["sddmm"] = oracle.sddmm(p.row_ptr, p.col_idx, sv, p.A, p.B)
    if "fusedmm" in ops:
        refs["fusedmm"] = oracle.fusedmm(p.row_ptr, p.col_idx, sv, p.A, p.B, p.D)
    return refs


def run_family(b, p, d, refs, algo, ws, expect, null_values=False):
    """Runs the ops in `refs` with one algo value on one workspace and checks every element."""
    sv = None if null_values else d.values
    worst = {}
    for op, (ref, T) in refs.items():
        if op == "spmm":
            out = torch.full((p.M, p.N), float("nan"), device="cuda")
            b.spmm(d.row_ptr, d.col_idx, d.values, d.D, K=p.K, out=out, workspace=ws, algo=algo)
            idx = b.OP_SPMM
        elif op == "sddmm":
            out = torch.full((p.nnz,), float("nan"), device="cuda")
            b.sddmm(d.row_ptr, d.col_idx, sv, d.A, d.B, out=out, workspace=ws, algo=algo)
            idx = b.OP_SDDMM
        else:
            out = torch.full((p.M, p.N), float("nan"), device="cuda")
            b.fusedmm(d.row_ptr, d.col_idx, sv, d.A, d.B, d.D, out=out, workspace=ws, algo=algo)
            idx = b.OP_FUSEDMM
        if expect is not None:
            assert b.last_algo(idx) == expect, f"{op} algo={algo} on {p.name} ran family {b.last_algo(idx)}"
        assert b.device_status(ws) == 0, f"{op} algo={algo} on {p.name}: a bounded device-side wait gave up"
        worst[op] = gate(out, ref, T, f"{op} algo={algo} {p.name}")
        del out
    return worst


def check_every_family(b, p, ops=OPS, null_values=False, families=(ROW, TILE, PREPARED)):
    d = DevProblem(p)
    refs = oracle_refs(p, ops, null_values)
    ws = torch.empty(max(b.workspace_bytes(i, p.M, p.K, p.Kd, p.N, p.nnz) for i in range(3)),
                     dtype=torch.uint8, device="cuda")
    if ROW in families:
        run_family(b, p, d, refs, ROW, ws, ROW, null_values)
    if TILE in families:
        run_family(b, p, d, refs, TILE, ws, TILE, null_values)
    if PREPARED in families:
        b.prepare_pattern(d.row_ptr, d.col_idx, p.K, ws)      # one table ...
        run_family(b, p, d, refs, PREPARED, ws, TILE, null_values)   # ... shared by the three ops
        run_family(b, p, d, refs, PREPARED, ws, TILE, null_values)   # and still intact afterwards
    torch.cuda.synchronize()
    assert d.pattern_untouched(), "row_ptr / col_idx changed"


@pytest.mark.parametrize("N", [128, 256, 512])
@pytest.mark.parametrize("density", [0.1, 0.2, 0.3])
def test_sweep_point_every_element(b, density, N):
    p = W.sweep_case(density, N)
    assert p.nnz == round(density * 8192 * 8192)
    check_every_family(b, p)


def test_sweep_point_automatic_choice(b):
    """What a caller gets without asking for a family: the dense-tile kernels at these densities."""
    p = W.sweep_case(0.3, 128)
    d = DevProblem(p)
    refs = oracle_refs(p, OPS)
    ws = torch.empty(max(b.workspace_bytes(i, p.M, p.K, p.Kd, p.N, p.nnz) for i in range(3)),
                     dtype=torch.uint8, device="cuda")
    run_family(b, p, d, refs, 0, ws, TILE)
    assert d.pattern_untouched()


@pytest.mark.parametrize("problem", range(8))
def test_attention_problem_every_element(b, problem):
    p = W.attention_case(problem)
    assert abs(p.nnz / 4096 ** 2 - 0.20) < 0.002
    check_every_family(b, p)
    if problem == 0:   # values all 1.0: the NULL form must give the same
        check_every_family(b, p, ops=("sddmm", "fusedmm"), null_values=True, families=(ROW, TILE))


def test_spmm_and_sddmm_configs_every_family(b):
    check_every_family(b, W.spmm_case(), ops=("spmm",))
    check_every_family(b, W.sddmm_case(), ops=("sddmm",))
    check_every_family(b, W.sddmm_case(), ops=("sddmm",), null_values=True, families=(ROW, TILE))


@pytest.mark.parametrize("name", [
    "grid_3k_1k_32_70",      # rectangular, width 32
    "grid_24k_8k_32_90",     # 192 row tiles (more than one per SM: the tile kernel's grid takes two waves), width 32
    "grid_24k_8k_128_90",    # the same at width 128
    "grid_32k_8k_128_80",    # 256 row tiles
    "grid_12k_4k_128_70",    # 96 row tiles, one K split
])
def test_paper_grid_case_every_element(b, name):
    p = W.paper_grid_case(name)
    check_every_family(b, p)
