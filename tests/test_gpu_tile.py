"""Parity of the dense-tile (tensor-core, 3xTF32) family against the CPU oracle, through the C ABI.
Same gate as the row family: |gpu - ref| <= 1e-5 * T + 1e-6 elementwise."""
import numpy as np
import pytest
import torch

import oracle
from paper_2311_00368_b200 import workloads as W
from tests.test_gpu_parity import DevProblem, _custom_rows, gate

pytestmark = pytest.mark.gpu

TILE, PREPARED = 3, 4


@pytest.fixture(scope="module")
def b():
    assert torch.cuda.is_available()
    from paper_2311_00368_b200 import binding
    return binding


def _ws(b, op, p):
    n = b.workspace_bytes(op, p.M, p.K, p.Kd, p.N, p.nnz)
    big = max(n, 64 << 20)
    return torch.empty(big, dtype=torch.uint8, device="cuda")


def spmm_tile_check(b, p, expect_algo=TILE):
    d = DevProblem(p)
    ws = _ws(b, b.OP_SPMM, p)
    ref, T = oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D)
    out = torch.full((p.M, p.N), float("nan"), device="cuda")
    b.spmm(d.row_ptr, d.col_idx, d.values, d.D, K=p.K, out=out, workspace=ws, algo=TILE)
    assert b.last_algo(b.OP_SPMM) == expect_algo
    assert b.device_status(ws) == 0, "a bounded wait inside the tile kernel gave up"
    r = gate(out, ref, T, f"spmm tile {p.name} M={p.M} K={p.K} N={p.N}")
    assert d.pattern_untouched()
    return r


@pytest.mark.parametrize("M,K,density,N,kind", [
    (256, 256, 0.10, 64, "uniform"),     # tiny-config shape
    (128, 128, 0.30, 32, "uniform"),     # one tile, one column group
    (257, 333, 0.30, 128, "uniform"),    # ragged M and K (K not a multiple of 32)
    (300, 512, 0.20, 100, "uniform"),    # N padded to 128 inside the scratch copy
    (130, 1024, 0.25, 644, "uniform"),   # TN = 256, three column tiles, ragged last one
    (512, 2048, 0.10, 256, "uniform"),   # several K splits
    (384, 1024, 0.20, 256, "powerlaw"),  # skewed rows incl. full rows
    (256, 512, 0.20, 128, "band"),
    (200, 640, 0.05, 36, "uniform"),     # sparse windows (8 lanes per row), N = 36
    (260, 700, 0.20, 63, "uniform"),     # widest output that still takes 64-column O tiles (odd: no TMA flush)
    (260, 700, 0.20, 65, "uniform"),     # narrowest output on 128-column O tiles
])
def test_spmm_tile_shapes(b, M, K, density, N, kind):
    p = W.small_random(2000 + M + N, M, K, density, 0, N, kind=kind)
    spmm_tile_check(b, p)


def test_spmm_tile_row_edges(b):
    lens = [0, 1, 31, 32, 33, 0, 127, 128, 129, 255, 256, 257, 2048, 0, 2, 64] * 9  # 144 rows
    p = _custom_rows(lens, 2048, 15, Kd=0, N=128)
    spmm_tile_check(b, p)


def test_spmm_tile_exact_on_small_integers(b):
    """Integers are exact in tf32 hi parts, so the tensor-core result must equal the exact one."""
    rng = np.random.default_rng(5)
    p = W.small_random(77, 256, 256, 0.3, 0, 64)
    p.values[:] = rng.integers(-4, 5, p.nnz).astype(np.float32)
    p.D[:] = rng.integers(-8, 9, p.D.shape).astype(np.float32)
    d = DevProblem(p)
    ws = _ws(b, b.OP_SPMM, p)
    out = b.spmm(d.row_ptr, d.col_idx, d.values, d.D, workspace=ws, algo=TILE)
    ref, _ = oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D)
    assert np.array_equal(out.cpu().numpy().astype(np.float64), ref)


def test_spmm_tile_falls_back_on_unsorted_rows(b):
    """Rows that are not strictly increasing are detected by the pre-pass on the device; the row
    kernels then produce the result within the same call."""
    p = W.small_random(91, 256, 300, 0.3, 0, 128)
    rng = np.random.default_rng(3)
    ci, v = p.col_idx.copy(), p.values.copy()
    a, e = p.row_ptr[5], p.row_ptr[6]
    perm = a + rng.permutation(e - a)
    ci[a:e], v[a:e] = ci[perm], v[perm]
    ci[p.row_ptr[9] + 1] = ci[p.row_ptr[9]]  # a duplicate in another row
    q = W.Problem("unsorted", p.M, p.K, p.row_ptr, ci, v, 0, p.N, None, None, p.D)
    spmm_tile_check(b, q)


def test_spmm_tile_hard_values(b):
    """Wide dynamic range: the hi/lo split must hold for tiny and large magnitudes alike."""
    p = W.small_random(123, 256, 512, 0.2, 0, 128)
    rng = np.random.default_rng(9)
    p.values[:] = (p.values * np.float32(10.0) ** rng.integers(-6, 7, p.nnz)).astype(np.float32)
    p.D[:] = (p.D * np.float32(10.0) ** rng.integers(-6, 7, p.D.shape)).astype(np.float32)
    spmm_tile_check(b, p)


def test_spmm_tile_config_and_auto(b):
    p = W.spmm_case()
    r = spmm_tile_check(b, p)
    assert r < 0.5  # 3xTF32 leaves a wide margin under the gate
    d = DevProblem(p)
    ws = _ws(b, b.OP_SPMM, p)
    out = b.spmm(d.row_ptr, d.col_idx, d.values, d.D, workspace=ws, algo=0)
    assert b.last_algo(b.OP_SPMM) == TILE  # 20% density: the planner picks the dense-tile family
    ref, T = oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D)
    gate(out, ref, T, "spmm auto")
    # a workspace that only fits the row family makes AUTO use the row family
    small = torch.empty(1 << 16, dtype=torch.uint8, device="cuda")
    out = b.spmm(d.row_ptr, d.col_idx, d.values, d.D, workspace=small, algo=0)
    assert b.last_algo(b.OP_SPMM) in (1, 2)   # the row family (natural order for few rows)
    gate(out, ref, T, "spmm auto, small workspace")
    with pytest.raises(b.B2spError) as e:
        b.spmm(d.row_ptr, d.col_idx, d.values, d.D, workspace=small, algo=TILE)
    assert e.value.status == 5


# ---- SDDMM and FusedMM on the dense-tile family -------------------------------------------------

def fused_tile_check(b, p, null_values=False, ops=("sddmm", "fusedmm")):
    d = DevProblem(p)
    sv_np = None if null_values else p.values
    sv = None if null_values else d.values
    worst = 0.0
    if "sddmm" in ops:
        ws = _ws(b, b.OP_SDDMM, p)
        ref, T = oracle.sddmm(p.row_ptr, p.col_idx, sv_np, p.A, p.B)
        out = torch.full((p.nnz,), float("nan"), device="cuda")
        b.sddmm(d.row_ptr, d.col_idx, sv, d.A, d.B, out=out, workspace=ws, algo=TILE)
        assert b.last_algo(b.OP_SDDMM) == TILE
        assert b.device_status(ws) == 0, "a bounded wait inside the SDDMM tile kernel gave up"
        worst = max(worst, gate(out, ref, T, f"sddmm tile {p.name} M={p.M} K={p.K} Kd={p.Kd}"))
    if "fusedmm" in ops:
        ws = _ws(b, b.OP_FUSEDMM, p)
        ref, T = oracle.fusedmm(p.row_ptr, p.col_idx, sv_np, p.A, p.B, p.D)
        out = torch.full((p.M, p.N), float("nan"), device="cuda")
        b.fusedmm(d.row_ptr, d.col_idx, sv, d.A, d.B, d.D, out=out, workspace=ws, algo=TILE)
        assert b.last_algo(b.OP_FUSEDMM) == TILE
        assert b.device_status(ws) == 0, "a bounded wait inside the FusedMM tile kernel gave up"
        worst = max(worst, gate(out, ref, T, f"fusedmm tile {p.name} M={p.M} K={p.K} Kd={p.Kd} N={p.N}"))
    assert d.pattern_untouched()
    return worst


@pytest.mark.parametrize("M,K,density,Kd,N,kind", [
    (128, 128, 0.30, 32, 32, "uniform"),      # one tile, one window group, smallest Kd
    (256, 256, 0.10, 64, 64, "uniform"),      # tiny-config shape
    (257, 333, 0.30, 128, 128, "uniform"),    # ragged M and K
    (300, 512, 0.20, 100, 100, "uniform"),    # Kd and N padded inside the scratch copies
    (130, 1024, 0.25, 20, 300, "uniform"),    # three O column tiles, small Kd
    (512, 2048, 0.10, 128, 256, "uniform"),   # several K splits, two column tiles
    (384, 1024, 0.20, 64, 128, "powerlaw"),   # skewed rows incl. full rows
    (256, 512, 0.20, 64, 64, "band"),
    (200, 640, 0.05, 36, 36, "uniform"),
    (260, 700, 0.20, 48, 64, "powerlaw"),     # 64-column O tile, several K splits
    (260, 700, 0.20, 48, 68, "powerlaw"),     # 128-column O tile just above the switch
])
def test_fused_and_sddmm_tile_shapes(b, M, K, density, Kd, N, kind):
    p = W.small_random(3000 + M + N, M, K, density, Kd, N, kind=kind)
    fused_tile_check(b, p)
    fused_tile_check(b, p, null_values=True)


def test_fused_tile_exact_on_small_integers(b):
    rng = np.random.default_rng(6)
    p = W.small_random(78, 256, 256, 0.3, 32, 64)
    p.values[:] = rng.integers(-2, 3, p.nnz).astype(np.float32)
    p.A[:] = rng.integers(-3, 4, p.A.shape).astype(np.float32)
    p.B[:] = rng.integers(-3, 4, p.B.shape).astype(np.float32)
    p.D[:] = rng.integers(-4, 5, p.D.shape).astype(np.float32)
    d = DevProblem(p)
    C = b.sddmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, workspace=_ws(b, b.OP_SDDMM, p), algo=TILE)
    ref, _ = oracle.sddmm(p.row_ptr, p.col_idx, p.values, p.A, p.B)
    assert np.array_equal(C.cpu().numpy().astype(np.float64), ref)
    O = b.fusedmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, d.D, workspace=_ws(b, b.OP_FUSEDMM, p), algo=TILE)
    ref, _ = oracle.fusedmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D)
    assert np.array_equal(O.cpu().numpy().astype(np.float64), ref)


def test_fused_tile_row_edges_and_inplace_sddmm(b):
    lens = [0, 1, 31, 32, 33, 0, 127, 128, 129, 255, 256, 257, 2048, 0, 2, 64] * 9
    p = _custom_rows(lens, 2048, 16, Kd=64, N=128)
    fused_tile_check(b, p)
    d = DevProblem(p)
    ref, T = oracle.sddmm(p.row_ptr, p.col_idx, p.values, p.A, p.B)
    vals = d.values.clone()
    b.sddmm(d.row_ptr, d.col_idx, vals, d.A, d.B, out=vals, workspace=_ws(b, b.OP_SDDMM, p), algo=TILE)
    gate(vals, ref, T, "sddmm tile in place")


def test_fused_tile_falls_back_on_unsorted_rows_and_large_kd(b):
    p = W.small_random(92, 256, 300, 0.3, 64, 128)
    rng = np.random.default_rng(4)
    ci, v = p.col_idx.copy(), p.values.copy()
    a, e = p.row_ptr[7], p.row_ptr[8]
    perm = a + rng.permutation(e - a)
    ci[a:e], v[a:e] = ci[perm], v[perm]
    q = W.Problem("unsorted", p.M, p.K, p.row_ptr, ci, v, p.Kd, p.N, p.A, p.B, p.D)
    fused_tile_check(b, q)
    # Kd > 128 is outside the tile family: an explicit request is refused, AUTO uses the row kernels
    big = W.small_random(93, 256, 256, 0.2, 160, 64)
    d = DevProblem(big)
    ws = torch.empty(64 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(b.B2spError) as e:
        b.fusedmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, d.D, workspace=ws, algo=TILE)
    assert e.value.status == 2
    out = b.fusedmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, d.D, workspace=ws, algo=0)
    assert b.last_algo(b.OP_FUSEDMM) in (1, 2)
    ref, T = oracle.fusedmm(big.row_ptr, big.col_idx, big.values, big.A, big.B, big.D)
    gate(out, ref, T, "fusedmm auto, Kd=160")


def test_fused_tile_configs(b):
    p = W.sddmm_case()
    d = DevProblem(p)
    ws = _ws(b, b.OP_SDDMM, p)
    ref, T = oracle.sddmm(p.row_ptr, p.col_idx, p.values, p.A, p.B)
    out = b.sddmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, workspace=ws, algo=TILE)
    assert b.last_algo(b.OP_SDDMM) == TILE and b.device_status(ws) == 0
    assert gate(out, ref, T, "sddmm config, tile") < 0.5
    out = b.sddmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, workspace=ws, algo=0)
    assert b.last_algo(b.OP_SDDMM) == TILE   # 10% density at 4096^2: past the measured cross-over
    assert b.device_status(ws) == 0
    gate(out, ref, T, "sddmm config, auto")
    p = W.attention_case(3)
    d = DevProblem(p)
    ws = _ws(b, b.OP_FUSEDMM, p)
    out = b.fusedmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, d.D, workspace=ws, algo=0)
    assert b.last_algo(b.OP_FUSEDMM) == TILE and b.device_status(ws) == 0
    rows = (0, 37, 2048, 4095)
    for r in rows:
        ref, T = oracle.fusedmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D, rows=(r, r + 1))
        ok, ratio = oracle.within_tolerance(out[r:r + 1].cpu().numpy(), ref, T)
        assert ok, f"attention row {r}: {ratio:.3g}"


# ---- prepared pattern ------------------------------------------------------------------------------

def test_prepared_pattern_is_shared_by_all_ops_and_stale_tables_are_detected(b):
    PREP = 4
    p = W.small_random(501, 300, 700, 0.25, 64, 128)
    d = DevProblem(p)
    n = max(b.workspace_bytes(op, p.M, p.K, p.Kd, p.N, p.nnz) for op in range(3))
    ws = torch.empty(max(n, 1 << 20), dtype=torch.uint8, device="cuda")
    b.prepare_pattern(d.row_ptr, d.col_idx, p.K, ws)
    refs = {"spmm": oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D),
            "sddmm": oracle.sddmm(p.row_ptr, p.col_idx, p.values, p.A, p.B),
            "fusedmm": oracle.fusedmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D)}

    def run_all(tag):
        for _ in range(2):   # the table survives repeated use by all three ops
            out = b.spmm(d.row_ptr, d.col_idx, d.values, d.D, workspace=ws, algo=PREP)
            gate(out, *refs["spmm"], f"spmm prepared {tag}")
            out = b.sddmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, workspace=ws, algo=PREP)
            gate(out, *refs["sddmm"], f"sddmm prepared {tag}")
            out = b.fusedmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, d.D, workspace=ws, algo=PREP)
            gate(out, *refs["fusedmm"], f"fusedmm prepared {tag}")
            assert b.device_status(ws) == 0

    run_all("fresh")
    # a workspace prepared for another matrix must not be trusted: the result stays correct
    q = W.small_random(502, 300, 700, 0.25, 64, 128)
    dq = DevProblem(q)
    b.prepare_pattern(dq.row_ptr, dq.col_idx, q.K, ws)
    run_all("stale table")
    # neither must a workspace that was never prepared (garbage header)
    ws.fill_(0x5a)
    run_all("garbage workspace")
    # nor one whose header a row-family call has rewritten
    b.prepare_pattern(d.row_ptr, d.col_idx, p.K, ws)
    b.spmm(d.row_ptr, d.col_idx, d.values, d.D, workspace=ws, algo=1)
    run_all("after a row-family call")


@pytest.mark.parametrize("width", [100, 101])
@pytest.mark.parametrize("ks", [1, 2, 3])
def test_k_split_epilogues(b, ks, width):
    """One K split stores O, two splits add their tiles into a zero-filled O, more go through slabs
    and the fixed-order sum: all three must give the same result, also for a ragged width, an output
    whose rows are padded, and an output that held NaNs before the call; repeated calls are bit-equal."""
    b.debug_force_k_splits(ks)
    try:
        _k_split_epilogues(b, ks, width)
    finally:
        b.debug_force_k_splits(0)


def _k_split_epilogues(b, ks, width):
    p = W.small_random(4100 + ks, 300, 1024, 0.2, 48, width)
    d = DevProblem(p)
    ws = _ws(b, b.OP_FUSEDMM, p)
    ref_f, T_f = oracle.fusedmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D)
    ref_s, T_s = oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D)
    for name, ref, T, call in (
            ("fusedmm", ref_f, T_f, lambda o: b.fusedmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, d.D, out=o, workspace=ws, algo=TILE)),
            ("spmm", ref_s, T_s, lambda o: b.spmm(d.row_ptr, d.col_idx, d.values, d.D, K=p.K, out=o, workspace=ws, algo=TILE))):
        for pad in (12, 13, 3):                       # rows 16-byte aligned (TMA flush, unless the width is odd) or not (plain stores / atomics)
            padded = torch.full((p.M, p.N + pad), float("nan"), device="cuda")
            out = padded[:, :p.N]
            call(out)
            assert b.device_status(ws) == 0
            gate(out, ref, T, f"{name} tile, {ks} K split(s), rows padded by {pad}")
            assert torch.isnan(padded[:, p.N:]).all(), "the padding of the output rows was written"
        again = torch.full((p.M, p.N), float("nan"), device="cuda")
        call(again)
        assert torch.equal(again, out.contiguous()), f"{name}: two runs differ ({ks} K splits)"


@pytest.mark.parametrize("M,K,Kd,N,kind,density", [
    (256, 512, 32, 128, "uniform", 0.15),      # two row tiles, one granule each
    (1000, 2048, 128, 200, "uniform", 0.15),   # ragged last row tile, two column tiles (CTAs in groups of two), ragged width
    (130, 4096, 100, 300, "powerlaw", 0.15),   # three column tiles: 49 groups of three CTAs (FusedMM: two phases at this width)
    (700, 8192, 64, 64, "uniform", 0.15),      # six row tiles of sixteen granules, one per CTA: sixteen slabs per tile
    (6400, 2048, 64, 128, "uniform", 0.05),    # 200 granules on 148 CTAs: one or two each, segments end inside row tiles
    (25600, 512, 128, 64, "uniform", 0.05),    # 200 row tiles of one granule: CTAs with two whole tiles (two A tiles)
    (20000, 1024, 32, 200, "powerlaw", 0.04),  # 157 row tiles of two granules, groups of two CTAs: up to three segments
    (9000, 1536, 128, 128, "band", 0.05),      # 71 row tiles of three granules
])
def test_balanced_partition_matches_plain(b, M, K, Kd, N, kind, density):
    """SPMM, SDDMM and FusedMM on the balanced partition (granules of all row tiles dealt evenly to the CTAs; SPMM and
    FusedMM: a slab per segment, the slab-sum kernel behind; FusedMM and SDDMM reload their A tile between segments)
    against the oracle, for bfloat16 operands too, on an output whose rows are padded and held NaNs; twice, bit-equal; and
    the plain partition the same way."""
    p = W.small_random(4300 + M, M, K, density, Kd, N, kind=kind)
    d = DevProblem(p)
    A16, B16, D16 = (t.to(torch.bfloat16) for t in (d.A, d.B, d.D))
    h = lambda t: t.float().cpu().numpy()
    calls = {
        "spmm": (oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D), oracle.spmm(p.row_ptr, p.col_idx, p.values, h(D16)),
                 lambda o, ws, algo: b.spmm(d.row_ptr, d.col_idx, d.values, d.D, K=p.K, out=o, workspace=ws, algo=algo),
                 lambda o, ws, algo: b.spmm(d.row_ptr, d.col_idx, d.values, D16, K=p.K, out=o, workspace=ws, algo=algo, dtype=torch.bfloat16),
                 b.OP_SPMM),
        "sddmm": (oracle.sddmm(p.row_ptr, p.col_idx, p.values, p.A, p.B), oracle.sddmm(p.row_ptr, p.col_idx, p.values, h(A16), h(B16)),
                  lambda o, ws, algo: b.sddmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, out=o, workspace=ws, algo=algo),
                  lambda o, ws, algo: b.sddmm(d.row_ptr, d.col_idx, d.values, A16, B16, out=o, workspace=ws, algo=algo, dtype=torch.bfloat16),
                  b.OP_SDDMM),
        "fusedmm": (oracle.fusedmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D),
                    oracle.fusedmm(p.row_ptr, p.col_idx, p.values, h(A16), h(B16), h(D16)),
                    lambda o, ws, algo: b.fusedmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, d.D, out=o, workspace=ws, algo=algo),
                    lambda o, ws, algo: b.fusedmm(d.row_ptr, d.col_idx, d.values, A16, B16, D16, out=o, workspace=ws, algo=algo, dtype=torch.bfloat16),
                    b.OP_FUSEDMM),
    }
    for part in (2, 1):
        b.debug_force_partition(part)
        try:
            ws = _ws(b, b.OP_FUSEDMM, p)
            b.prepare_pattern(d.row_ptr, d.col_idx, p.K, ws)
            for name, ((ref, T), (ref16, T16), call, call16, op) in calls.items():
                shape = (p.nnz,) if name == "sddmm" else (p.M, p.N)
                for pad in (4, 3):
                    if name == "sddmm":
                        out = torch.full(shape, float("nan"), device="cuda")
                    else:
                        padded = torch.full((p.M, p.N + pad), float("nan"), device="cuda")
                        out = padded[:, :p.N]
                    call(out, ws, PREPARED)
                    assert b.last_algo(op) == TILE and b.device_status(ws) == 0
                    gate(out, ref, T, f"{name} partition {part}, rows padded by {pad}")
                    if name != "sddmm":
                        assert torch.isnan(padded[:, p.N:]).all(), "the padding of the output rows was written"
                again = torch.full(shape, float("nan"), device="cuda")
                call(again, ws, TILE)
                assert torch.equal(again, out.contiguous()), f"{name}: two runs differ (partition {part})"
                o16 = torch.full(shape, float("nan"), device="cuda")
                call16(o16, ws, TILE)
                assert b.device_status(ws) == 0
                gate(o16, ref16, T16, f"{name} bf16 partition {part}")
        finally:
            b.debug_force_partition(0)
    assert d.pattern_untouched()


def test_balanced_partition_falls_back_on_non_finite_operand(b):
    """The slab-sum kernel must not touch O when the row kernels produced it (a NaN in an unreferenced row of D)."""
    p = W.small_random(4400, 600, 2048, 0.2, 32, 128)
    keep = p.col_idx != 9
    lens = np.add.reduceat(keep.astype(np.int64), p.row_ptr[:-1].astype(np.int64))
    rp = np.zeros(p.M + 1, dtype=np.int32)
    rp[1:] = np.cumsum(lens)
    q = W.Problem("hole", p.M, p.K, rp, p.col_idx[keep], p.values[keep], p.Kd, p.N, p.A, p.B, p.D.copy())
    ref, T = oracle.spmm(q.row_ptr, q.col_idx, q.values, q.D)
    d = DevProblem(q)
    d.D[9, :] = float("nan")
    b.debug_force_partition(2)
    try:
        ws = _ws(b, b.OP_SPMM, q)
        for _ in range(2):
            out = torch.full((q.M, q.N), float("nan"), device="cuda")
            b.spmm(d.row_ptr, d.col_idx, d.values, d.D, K=q.K, out=out, workspace=ws, algo=TILE)
            assert b.device_status(ws) == 0
            gate(out, ref, T, "spmm, balanced partition, NaN in an unreferenced row of D")
    finally:
        b.debug_force_partition(0)


def test_tile_accuracy_on_same_sign_data_and_long_rows(b):
    """The tensor core adds into its fp32 accumulator with truncation, a bias that grows with the
    number of MMAs per output; on same-sign data nothing cancels it.  The planner caps the columns of
    S per K split, so the error must stay well inside the gate for K = 32768 as for K = 8192."""
    for M, K in ((256, 8192), (128, 32768)):
        p = W.small_random(4200 + K, M, K, 0.3, 64, 128)
        rng = np.random.default_rng(5)
        p.values = rng.uniform(0.5, 1.5, p.nnz).astype(np.float32)
        p.A = rng.uniform(0.5, 1.5, p.A.shape).astype(np.float32)
        p.B = rng.uniform(0.5, 1.5, p.B.shape).astype(np.float32)
        p.D = rng.uniform(0.5, 1.5, p.D.shape).astype(np.float32)
        assert spmm_tile_check(b, p) < 0.6
        assert fused_tile_check(b, p) < 0.6


def test_entry_points_can_be_captured_in_a_cuda_graph(b):
    """The device entry points only enqueue work (no allocation, no synchronisation), so a step of
    all three ops, row family and dense-tile family alike, can be captured once and replayed."""
    p = W.small_random(4300, 384, 1024, 0.2, 64, 128)
    d = DevProblem(p)
    ws = _ws(b, b.OP_FUSEDMM, p)
    O1 = torch.empty((p.M, p.N), device="cuda")
    O2 = torch.empty((p.M, p.N), device="cuda")
    C = torch.empty(p.nnz, device="cuda")
    refs = (oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D),
            oracle.sddmm(p.row_ptr, p.col_idx, p.values, p.A, p.B),
            oracle.fusedmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D))
    for algo in (TILE, 1):
        def step():
            b.spmm(d.row_ptr, d.col_idx, d.values, d.D, K=p.K, out=O1, workspace=ws, algo=algo)
            b.sddmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, out=C, workspace=ws, algo=algo)
            b.fusedmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, d.D, out=O2, workspace=ws, algo=algo)
        step()                                   # first use outside the capture (one-time driver queries)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            step()
        for out in (O1, O2, C):
            out.fill_(float("nan"))
        g.replay()
        torch.cuda.synchronize()
        assert b.device_status(ws) == 0
        for name, out, (ref, T) in zip(("spmm", "sddmm", "fusedmm"), (O1, C, O2), refs):
            gate(out, ref, T, f"{name} replayed from a CUDA graph, algo={algo}")


def test_non_finite_values_in_rows_nobody_refers_to(b):
    """Eq. 1-3 only touch the rows of B and D that a stored entry names.  The dense-tile kernels multiply
    whole windows (by zero where nothing is stored), so an Inf or NaN in an unreferenced row -- for instance
    uninitialised padding -- would leak into every output; the operand pre-pass detects non-finite values
    and the row kernels produce the result of that call.  The detection is per call: the next call on the
    same (prepared) workspace with clean operands runs on the tile kernels again."""
    p = W.small_random(4400, 300, 700, 0.2, 64, 128)
    dead = np.array([5, 77, 699])
    keep = ~np.isin(p.col_idx, dead)
    lens = np.add.reduceat(keep.astype(np.int64), p.row_ptr[:-1].astype(np.int64))
    rp = np.zeros(p.M + 1, dtype=np.int32)
    rp[1:] = np.cumsum(lens)
    q = W.Problem("holes", p.M, p.K, rp, p.col_idx[keep], p.values[keep], p.Kd, p.N, p.A.copy(), p.B.copy(), p.D.copy())
    refs = (oracle.spmm(q.row_ptr, q.col_idx, q.values, q.D),
            oracle.sddmm(q.row_ptr, q.col_idx, q.values, q.A, q.B),
            oracle.fusedmm(q.row_ptr, q.col_idx, q.values, q.A, q.B, q.D))
    dirty = W.Problem("holes", q.M, q.K, q.row_ptr, q.col_idx, q.values, q.Kd, q.N, q.A, q.B.copy(), q.D.copy())
    dirty.D[5, :] = np.nan
    dirty.D[699, 3] = np.inf
    dirty.B[77, :] = -np.inf
    dirty.B[5, 0] = np.nan
    ref_d = (oracle.spmm(dirty.row_ptr, dirty.col_idx, dirty.values, dirty.D),
             oracle.sddmm(dirty.row_ptr, dirty.col_idx, dirty.values, dirty.A, dirty.B),
             oracle.fusedmm(dirty.row_ptr, dirty.col_idx, dirty.values, dirty.A, dirty.B, dirty.D))
    for r_clean, r_dirty in zip(refs, ref_d):   # the oracle never reads those rows
        assert np.array_equal(r_clean[0], r_dirty[0]) and np.all(np.isfinite(r_dirty[0]))
    dc, dd = DevProblem(q), DevProblem(dirty)
    n = max(b.workspace_bytes(op, q.M, q.K, q.Kd, q.N, q.nnz) for op in range(3))
    ws = torch.empty(max(n, 1 << 20), dtype=torch.uint8, device="cuda")

    def run(d, algo, tag):
        out = b.spmm(d.row_ptr, d.col_idx, d.values, d.D, workspace=ws, algo=algo)
        gate(out, *refs[0], f"spmm {tag}")
        out = b.sddmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, workspace=ws, algo=algo)
        gate(out, *refs[1], f"sddmm {tag}")
        out = b.fusedmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, d.D, workspace=ws, algo=algo)
        gate(out, *refs[2], f"fusedmm {tag}")
        assert b.device_status(ws) == 0
        flags = ws[320:332].view(torch.int32).cpu().numpy()
        assert flags[1] == 0 and flags[2] == 0, "the per-call flag and its reader count are reset by the fallback"
        return int(flags[0])

    run(dd, TILE, "tile, NaN / Inf in unreferenced rows")
    run(dc, TILE, "tile, clean operands afterwards")
    b.prepare_pattern(dc.row_ptr, dc.col_idx, q.K, ws)
    assert run(dc, 4, "prepared table, clean") == 0
    b.prepare_pattern(dd.row_ptr, dd.col_idx, q.K, ws)
    assert run(dd, 4, "prepared table, NaN / Inf in unreferenced rows") == 0   # the table itself stays usable
    b.prepare_pattern(dc.row_ptr, dc.col_idx, q.K, ws)
    assert run(dc, 4, "prepared table, clean again") == 0
    # a row of A without stored entries may hold anything as well
    lens = np.diff(q.row_ptr)
    empty = W.Problem("empty-row", q.M, q.K, q.row_ptr.copy(), q.col_idx, q.values, q.Kd, q.N, q.A.copy(), q.B, q.D)
    a, e = empty.row_ptr[10], empty.row_ptr[11]
    ci = np.concatenate([q.col_idx[:a], q.col_idx[e:]])
    v = np.concatenate([q.values[:a], q.values[e:]])
    empty.row_ptr[11:] -= (e - a)
    empty = W.Problem("empty-row", q.M, q.K, empty.row_ptr, ci, v, q.Kd, q.N, empty.A, q.B, q.D)
    empty.A[10, :] = np.nan
    de = DevProblem(empty)
    ref, T = oracle.fusedmm(empty.row_ptr, empty.col_idx, empty.values, empty.A, empty.B, empty.D)
    assert np.all(ref[10] == 0) and np.all(np.isfinite(ref))
    out = b.fusedmm(de.row_ptr, de.col_idx, de.values, de.A, de.B, de.D, workspace=ws, algo=TILE)
    gate(out, ref, T, "fusedmm tile, NaN in the A row of an empty row of S")


def test_a_wait_that_runs_out_is_reported_and_the_gpu_stays_usable(b):
    """Every wait inside the dense-tile kernels is bounded.  The debug hook withholds one operand chunk in every
    CTA and shortens the limit to 2 ms: the waits run out, the CTAs leave through their normal teardown, the
    status word says B2SP_ERR_TIMEOUT (6) -- through b2sp_device_status and through the host-buffer form -- and the
    next call on the same workspace is correct again."""
    p = W.small_random(4500, 384, 1024, 0.2, 64, 128)
    d = DevProblem(p)
    ws = _ws(b, b.OP_FUSEDMM, p)
    big = W.spmm_case()     # large enough for the host form's automatic choice to be the dense-tile family
    t = lambda x: torch.from_numpy(x).pin_memory()
    hO = torch.empty((big.M, big.N), dtype=torch.float32).pin_memory()
    b.debug_inject_wait_timeout(1, 2_000_000)
    try:
        b.spmm(d.row_ptr, d.col_idx, d.values, d.D, workspace=ws, algo=TILE)
        assert b.device_status(ws) == 6
        b.sddmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, workspace=ws, algo=TILE)
        assert b.device_status(ws) == 6
        b.fusedmm(d.row_ptr, d.col_idx, d.values, d.A, d.B, d.D, workspace=ws, algo=TILE)
        assert b.device_status(ws) == 6
        with pytest.raises(b.B2spError) as e:
            b.spmm_host(t(big.row_ptr), t(big.col_idx), t(big.values), t(big.D), hO)
        assert e.value.status == 6
    finally:
        b.debug_inject_wait_timeout(-1)
    torch.cuda.synchronize()
    spmm_tile_check(b, p)
    fused_tile_check(b, p)
    ref, T = oracle.spmm(big.row_ptr, big.col_idx, big.values, big.D)
    gate(b.spmm_host(t(big.row_ptr), t(big.col_idx), t(big.values), t(big.D), hO), ref, T, "spmm_host after the hook")


def test_l2_pull_probe(b):
    """The measurement aid behind bench.py's `roofline.l2_operand_stream`: a plausible rate, and the argument checks."""
    per_sm, total = b.probe_l2_pull()
    assert 20.0 < per_sm < 500.0 and 50.0 * per_sm < total < 400.0 * per_sm
    import ctypes
    small = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    x, y = ctypes.c_double(), ctypes.c_double()
    assert b.lib.b2sp_probe_l2_pull(small.data_ptr(), small.numel(), ctypes.byref(x), ctypes.byref(y), None) == 1
