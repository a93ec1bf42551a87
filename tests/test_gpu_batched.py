"""b2sp_fusedmm_batched: a batch of independent FusedMM problems of the same sizes in one call, checked
problem by problem and element by element against the CPU oracle (gate |gpu - ref| <= 1e-5 * T + 1e-6).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2311_00368_b200 import workloads as W
from tests.test_gpu_parity import gate

pytestmark = pytest.mark.gpu

ROW, TILE, PREPARED = 1, 3, 4


@pytest.fixture(scope="module")
def b():
    assert torch.cuda.is_available()
    from paper_2311_00368_b200 import binding
    return binding


class Stacked:
    """The problems' CSR arrays padded to a common length and stacked, the dense operands stacked."""

    def __init__(self, problems, pad_to=4):
        self.problems = problems
        nb, p0 = len(problems), problems[0]
        stride = max(p.nnz for p in problems)
        stride = (stride + pad_to - 1) // pad_to * pad_to
        rp = np.stack([p.row_ptr for p in problems])
        ci = np.zeros((nb, stride), dtype=np.int32)
        sv = np.full((nb, stride), np.nan, dtype=np.float32)      # the padding is never read
        for i, p in enumerate(problems):
            ci[i, :p.nnz], sv[i, :p.nnz] = p.col_idx, p.values
        t = lambda x: torch.from_numpy(np.ascontiguousarray(x)).cuda()
        self.row_ptr, self.col_idx, self.values = t(rp), t(ci), t(sv)
        self.A = t(np.stack([p.A for p in problems]))
        self.B = t(np.stack([p.B for p in problems]))
        self.D = t(np.stack([p.D for p in problems]))
        self.nb, self.M, self.K, self.Kd, self.N, self.stride = nb, p0.M, p0.K, p0.Kd, p0.N, stride
        self._rp0, self._ci0 = self.row_ptr.clone(), self.col_idx.clone()
        self.refs = [oracle.fusedmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D) for p in problems]
        self.refs_unit = None

    def workspace(self, b):
        n = b.workspace_bytes_batched(self.nb, self.M, self.K, self.Kd, self.N, self.stride)
        return torch.empty(max(n, 1 << 20), dtype=torch.uint8, device="cuda")

    def check(self, out, what, refs=None):
        worst = 0.0
        for i, (ref, T) in enumerate(refs or self.refs):
            worst = max(worst, gate(out[i], ref, T, f"{what}, problem {i}"))
        assert torch.equal(self.row_ptr, self._rp0) and torch.equal(self.col_idx, self._ci0), "pattern arrays changed"
        return worst


def run(b, s, algo, ws, expect, what, values=True, out=None):
    if out is None:
        out = torch.full((s.nb, s.M, s.N), float("nan"), device="cuda")
    b.fusedmm_batched(s.row_ptr, s.col_idx, s.values if values else None, s.A, s.B, s.D, out=out, workspace=ws, algo=algo)
    assert b.last_algo(b.OP_FUSEDMM) == expect, f"{what}: ran family {b.last_algo(b.OP_FUSEDMM)}"
    assert b.device_status(ws) == 0, f"{what}: a bounded device-side wait gave up"
    return out


@pytest.mark.parametrize("M,K,Kd,N,kind", [
    (300, 700, 48, 100, "uniform"),      # ragged tiles, padded widths
    (256, 512, 64, 64, "band"),          # 64-column O tiles
    (130, 1024, 20, 260, "powerlaw"),    # wider than 256 columns: the row kernels only
    (257, 333, 128, 63, "uniform"),      # odd width: plain stores in the flush
])
def test_small_batches_every_family(b, M, K, Kd, N, kind):
    probs = [W.small_random(5000 + 10 * i + M, M, K, d, Kd, N, kind=kind) for i, d in enumerate((0.2, 0.05, 0.3))]
    s = Stacked(probs)
    ws = s.workspace(b)
    tile_ok = N <= 256
    s.check(run(b, s, ROW, ws, 2, "row family"), "batched, row family")
    if tile_ok:
        s.check(run(b, s, TILE, ws, TILE, "tile"), "batched, dense-tile family")
        b.prepare_pattern_batched(s.row_ptr, s.col_idx, K, ws)
        for _ in range(2):
            s.check(run(b, s, PREPARED, ws, TILE, "prepared"), "batched, prepared tables")
    else:
        with pytest.raises(b.B2spError) as e:
            run(b, s, TILE, ws, TILE, "tile")
        assert e.value.status == 2
    # all-ones sampling pattern (s_values = NULL)
    refs = [oracle.fusedmm(p.row_ptr, p.col_idx, None, p.A, p.B, p.D) for p in probs]
    s.check(run(b, s, TILE if tile_ok else ROW, ws, TILE if tile_ok else 2, "NULL values", values=False),
            "batched, NULL values", refs)


@pytest.mark.parametrize("ks", [2, 3])
def test_batch_with_several_k_splits(b, ks):
    """Slabs, arrival counters and the fixed-order sum are per problem."""
    probs = [W.small_random(5100 + i, 300, 1024, 0.2, 48, 100) for i in range(3)]
    s = Stacked(probs)
    b.debug_force_k_splits(ks)
    try:
        ws = s.workspace(b)
        padded = torch.full((s.nb, s.M + 3, s.N + 12), float("nan"), device="cuda")
        out = padded[:, :s.M, :s.N]
        run(b, s, TILE, ws, TILE, f"{ks} K splits", out=out)
        s.check(out, f"batched, {ks} K splits")
        assert torch.isnan(padded[:, s.M:, :]).all() and torch.isnan(padded[:, :, s.N:]).all(), "padding written"
        again = run(b, s, TILE, ws, TILE, f"{ks} K splits, again")
        assert torch.equal(again, out.contiguous()), "two runs differ"
    finally:
        b.debug_force_k_splits(0)


@pytest.mark.parametrize("nb,M,K,Kd,N", [
    (3, 300, 1024, 48, 100),     # three row tiles of two granules per problem
    (5, 4100, 1024, 64, 64),     # 33 row tiles per problem: 330 granules on 148 CTAs, segments run from one problem into the next
    (2, 1500, 2048, 128, 200),   # two column tiles: groups of two CTAs
])
def test_batch_on_the_balanced_partition(b, nb, M, K, Kd, N):
    """The granules of all problems' row tiles dealt evenly to the CTAs: a segment names its problem (window table,
    stored values, operand rows, slab, output).  Against the oracle, NULL values and a shared pattern too, twice
    bit-equal, and the plain partition the same way."""
    probs = [W.small_random(5600 + 7 * i + M, M, K, d, Kd, N) for i, d in zip(range(nb), (0.06, 0.03, 0.1, 0.05, 0.08))]
    s = Stacked(probs)
    refs_null = [oracle.fusedmm(p.row_ptr, p.col_idx, None, p.A, p.B, p.D) for p in probs]
    for part in (2, 1):
        b.debug_force_partition(part)
        try:
            ws = s.workspace(b)
            padded = torch.full((s.nb, s.M + 3, s.N + 12), float("nan"), device="cuda")
            out = padded[:, :s.M, :s.N]
            run(b, s, TILE, ws, TILE, f"partition {part}", out=out)
            s.check(out, f"batched, partition {part}")
            assert torch.isnan(padded[:, s.M:, :]).all() and torch.isnan(padded[:, :, s.N:]).all(), "padding written"
            b.prepare_pattern_batched(s.row_ptr, s.col_idx, K, ws)
            again = run(b, s, PREPARED, ws, TILE, f"partition {part}, prepared")
            assert torch.equal(again, out.contiguous()), "two runs differ"
            s.check(run(b, s, TILE, ws, TILE, "NULL values", values=False), f"batched, partition {part}, NULL values", refs_null)
            # one pattern for all problems (stride 0), operands per problem
            p0 = probs[0]
            t = lambda x: torch.from_numpy(np.ascontiguousarray(x)).cuda()
            shared = [oracle.fusedmm(p0.row_ptr, p0.col_idx, p0.values, p.A, p.B, p.D) for p in probs]
            o2 = torch.full((s.nb, s.M, s.N), float("nan"), device="cuda")
            b.fusedmm_batched(t(p0.row_ptr), t(p0.col_idx), t(p0.values), s.A, s.B, s.D, out=o2, workspace=ws, algo=TILE)
            assert b.last_algo(b.OP_FUSEDMM) == TILE and b.device_status(ws) == 0
            s.check(o2, f"batched, partition {part}, shared pattern", shared)
        finally:
            b.debug_force_partition(0)


def test_shared_pattern_and_shared_operands(b):
    """Stride 0: one pattern (1-D CSR arrays) and one D for all problems, A and B per problem."""
    p0 = W.small_random(5200, 260, 640, 0.2, 64, 128)
    rng = np.random.default_rng(7)
    probs = [W.Problem(f"shared{i}", p0.M, p0.K, p0.row_ptr, p0.col_idx, p0.values, p0.Kd, p0.N,
                       W.dense_normal(rng, p0.M, p0.Kd), W.dense_normal(rng, p0.K, p0.Kd), p0.D) for i in range(4)]
    s = Stacked(probs)
    t = lambda x: torch.from_numpy(np.ascontiguousarray(x)).cuda()
    rp, ci, sv, D = t(p0.row_ptr), t(p0.col_idx), t(p0.values), t(p0.D)
    ws = torch.empty(max(b.workspace_bytes_batched(4, p0.M, p0.K, p0.Kd, p0.N, p0.nnz), 1 << 20), dtype=torch.uint8, device="cuda")
    for algo, expect in ((TILE, TILE), (ROW, 2)):
        out = torch.full((4, p0.M, p0.N), float("nan"), device="cuda")
        b.fusedmm_batched(rp, ci, sv, s.A, s.B, D, out=out, workspace=ws, algo=algo)
        assert b.last_algo(b.OP_FUSEDMM) == expect and b.device_status(ws) == 0
        s.check(out, f"shared pattern, algo {algo}")


def test_batch_with_an_unsorted_problem_falls_back(b):
    probs = [W.small_random(5300 + i, 256, 300, 0.3, 64, 128) for i in range(3)]
    p = probs[1]
    rng = np.random.default_rng(4)
    ci, v = p.col_idx.copy(), p.values.copy()
    a, e = p.row_ptr[7], p.row_ptr[8]
    perm = a + rng.permutation(e - a)
    ci[a:e], v[a:e] = ci[perm], v[perm]
    probs[1] = W.Problem("unsorted", p.M, p.K, p.row_ptr, ci, v, p.Kd, p.N, p.A, p.B, p.D)
    s = Stacked(probs)
    ws = s.workspace(b)
    s.check(run(b, s, TILE, ws, TILE, "unsorted"), "batched, one problem with an unsorted row")


def test_argument_errors_batched(b):
    probs = [W.small_random(5400 + i, 64, 64, 0.3, 16, 16) for i in range(2)]
    s = Stacked(probs)
    ws = s.workspace(b)
    i, ll, vp = b.ctypes.c_int, b.ctypes.c_longlong, b.ctypes.c_void_p
    ptr = lambda t: vp(t.data_ptr())
    out = torch.empty((2, 64, 16), device="cuda")

    def call(batch=2, rps=65, so=64 * 16, algo=0):
        return b.lib.b2sp_fusedmm_batched(batch, 64, 64, 16, 16, s.stride, ptr(s.row_ptr), rps, ptr(s.col_idx),
                                          ptr(s.values), ptr(s.A), 16, 64 * 16, ptr(s.B), 16, 64 * 16, ptr(s.D), 16,
                                          64 * 16, ptr(out), 16, so, ptr(ws), ws.numel(), algo, None)
    assert call() == 0
    assert call(batch=0) == 1
    assert call(rps=10) == 1           # row pointer arrays would overlap
    assert call(so=100) == 1           # outputs would overlap
    assert call(algo=9) == 1


def test_attention_config_in_one_call(b):
    """The eight attention-shaped problems (4096 x 4096, band + random, 20%, head dim 64) in one call, every
    element of every output, on each family; the automatic choice is the dense-tile family."""
    probs = [W.attention_case(i) for i in range(8)]
    s = Stacked(probs)
    ws = s.workspace(b)
    s.check(run(b, s, 0, ws, TILE, "auto"), "attention batch, automatic choice")
    b.prepare_pattern_batched(s.row_ptr, s.col_idx, s.K, ws)
    w = s.check(run(b, s, PREPARED, ws, TILE, "prepared"), "attention batch, prepared tables")
    assert w < 0.5
    s.check(run(b, s, ROW, ws, 2, "row"), "attention batch, row family")


def test_batched_call_can_be_captured_in_a_cuda_graph(b):
    """The batched entry point only enqueues work; a captured call replays correctly on new contents of O."""
    probs = [W.small_random(5500 + i, 384, 1024, 0.2, 64, 128) for i in range(3)]
    s = Stacked(probs)
    ws = s.workspace(b)
    out = torch.full((s.nb, s.M, s.N), float("nan"), device="cuda")
    for algo, expect in ((TILE, TILE), (ROW, 2)):
        run(b, s, algo, ws, expect, "before the capture", out=out)      # one-time driver queries happen here
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            b.fusedmm_batched(s.row_ptr, s.col_idx, s.values, s.A, s.B, s.D, out=out, workspace=ws, algo=algo)
        out.fill_(float("nan"))
        g.replay()
        torch.cuda.synchronize()
        assert b.device_status(ws) == 0
        s.check(out, f"batched call replayed from a CUDA graph, algo {algo}")


def test_batched_bf16_operands(b):
    """b2sp_fusedmm_batched_bf16: bfloat16 A, B, D, fp32 accumulation; the oracle runs on the rounded values."""
    probs = [W.small_random(5600 + i, 300, 700, d, 64, 64, kind="uniform") for i, d in enumerate((0.2, 0.1, 0.3))]
    bf = lambda x: torch.from_numpy(np.ascontiguousarray(x)).to(torch.bfloat16)
    rounded = []
    for p in probs:
        A, B, D = bf(p.A), bf(p.B), bf(p.D)
        rounded.append(W.Problem(p.name, p.M, p.K, p.row_ptr, p.col_idx, p.values, p.Kd, p.N,
                                 A.float().numpy(), B.float().numpy(), D.float().numpy()))
    s = Stacked(rounded)            # references from the bf16-rounded operands
    A16, B16, D16 = s.A.to(torch.bfloat16), s.B.to(torch.bfloat16), s.D.to(torch.bfloat16)   # exact: already rounded
    ws = s.workspace(b)
    for algo, expect in ((TILE, TILE), (ROW, 2)):
        out = torch.full((s.nb, s.M, s.N), float("nan"), device="cuda")
        b.fusedmm_batched(s.row_ptr, s.col_idx, s.values, A16, B16, D16, out=out, workspace=ws, algo=algo,
                          dtype=torch.bfloat16)
        assert b.last_algo(b.OP_FUSEDMM) == expect and b.device_status(ws) == 0
        s.check(out, f"batched bf16, algo {algo}")
