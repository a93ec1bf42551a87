"""Seeded random shapes through every entry point and family: sizes that are not multiples of the tile, odd
widths, several densities and row-length laws, fp32 and bfloat16 operands, NULL values, batches of one to four
problems, prepared and stateless calls, either partition of the dense-tile work.  Everything is checked element by element against the CPU oracle
(|gpu - ref| <= 1e-5 * T + 1e-6) and the device status word must stay clear."""
import numpy as np
import pytest
import torch

import oracle
from paper_2311_00368_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _one_case(b, rng):
    dev = lambda x: torch.from_numpy(np.ascontiguousarray(x)).cuda()
    bf = lambda x: torch.from_numpy(np.ascontiguousarray(x)).to(torch.bfloat16)
    M, K = int(rng.integers(1, 600)), int(rng.integers(32, 1500))
    dens = float(rng.choice([0.05, 0.2, 0.4]))
    Kd = int(rng.choice([4, 8, 16, 32, 36, 64, 100, 128, 132]))
    N = int(rng.choice([4, 8, 32, 64, 100, 128, 132, 256, 300]))
    nb = int(rng.integers(1, 5))
    kind = str(rng.choice(["uniform", "powerlaw"]))
    probs = [W.small_random(int(rng.integers(1 << 30)), M, K, dens, Kd, N, kind=kind) for _ in range(nb)]
    if any(p.nnz == 0 for p in probs):
        return
    algo = int(rng.choice([0, 1, 3, 4]))
    use_bf, null = bool(rng.integers(0, 2)), bool(rng.random() < 0.25)
    part = int(rng.choice([0, 1, 2]))   # the dense-tile planner's partition: its choice, tiles x K splits, balanced
    what = f"M={M} K={K} d={dens} Kd={Kd} N={N} nb={nb} {kind} algo={algo} bf16={use_bf} null={null} partition={part}"
    b.debug_force_partition(part)
    try:
        _run_case(b, rng, M, K, Kd, N, nb, probs, algo, use_bf, null, what)
    finally:
        b.debug_force_partition(0)


def _run_case(b, rng, M, K, Kd, N, nb, probs, algo, use_bf, null, what):
    dev = lambda x: torch.from_numpy(np.ascontiguousarray(x)).cuda()
    bf = lambda x: torch.from_numpy(np.ascontiguousarray(x)).to(torch.bfloat16)
    if use_bf:                      # the bfloat16 values are the inputs: the oracle sees the rounded operands
        for p in probs:
            p.A, p.B, p.D = (bf(x).float().numpy() for x in (p.A, p.B, p.D))
    dt = torch.bfloat16 if use_bf else torch.float32
    cvt = (lambda x: dev(x).to(torch.bfloat16)) if use_bf else dev
    stride = (max(p.nnz for p in probs) + 3) // 4 * 4
    ci, sv = np.zeros((nb, stride), np.int32), np.zeros((nb, stride), np.float32)
    for i, p in enumerate(probs):
        ci[i, :p.nnz], sv[i, :p.nnz] = p.col_idx, p.values
    rp, cid, svd = dev(np.stack([p.row_ptr for p in probs])), dev(ci), (None if null else dev(sv))
    A, B, D = (cvt(np.stack([getattr(p, k) for p in probs])) for k in "ABD")

    def check(got, ref_T, tag):
        ok, ratio = oracle.within_tolerance(got.cpu().numpy(), *ref_T)
        assert ok, f"{tag}: {what}: worst error / allowed = {ratio:.3g}"

    # the batched call
    ws = torch.empty(max(b.workspace_bytes_batched(nb, M, K, Kd, N, stride), 1 << 20), dtype=torch.uint8, device="cuda")
    a = algo if (Kd <= 128 and N <= 256) or algo in (0, 1) else 1
    if a == 4:
        b.prepare_pattern_batched(rp, cid, K, ws)
    out = torch.full((nb, M, N), float("nan"), device="cuda")
    b.fusedmm_batched(rp, cid, svd, A, B, D, out=out, workspace=ws, algo=a, dtype=dt)
    assert b.device_status(ws) == 0, what
    for i, p in enumerate(probs):
        check(out[i], oracle.fusedmm(p.row_ptr, p.col_idx, None if null else p.values, p.A, p.B, p.D), f"batched, problem {i}")
    # the three single-problem ops on problem 0
    p = probs[0]
    w1 = torch.empty(max(max(b.workspace_bytes(o, M, K, Kd, N, p.nnz) for o in range(3)), 1 << 20), dtype=torch.uint8, device="cuda")
    a1 = algo if Kd <= 128 or algo in (0, 1) else 1
    r0, c0, v0 = dev(p.row_ptr), dev(p.col_idx), dev(p.values)
    if a1 == 4:
        b.prepare_pattern(r0, c0, K, w1)
    check(b.spmm(r0, c0, v0, D[0], K=K, workspace=w1, algo=a1, dtype=dt), oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D), "spmm")
    check(b.sddmm(r0, c0, None if null else v0, A[0], B[0], workspace=w1, algo=a1, dtype=dt),
          oracle.sddmm(p.row_ptr, p.col_idx, None if null else p.values, p.A, p.B), "sddmm")
    check(b.fusedmm(r0, c0, None if null else v0, A[0], B[0], D[0], workspace=w1, algo=a1, dtype=dt),
          oracle.fusedmm(p.row_ptr, p.col_idx, None if null else p.values, p.A, p.B, p.D), "fusedmm")
    assert b.device_status(w1) == 0, what
    assert torch.equal(r0.cpu(), torch.from_numpy(p.row_ptr)) and torch.equal(c0.cpu(), torch.from_numpy(p.col_idx)), what


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_shapes_every_entry_point(seed):
    assert torch.cuda.is_available()
    from paper_2311_00368_b200 import binding as b
    rng = np.random.default_rng(seed)
    for _ in range(25):
        _one_case(b, rng)


def test_random_large_shapes_on_the_balanced_partition():
    """Seeded shapes with tens to hundreds of row tiles, the dense-tile planner pinned to the balanced partition (several
    segments per CTA, groups of CTAs for wide outputs, A tiles reloaded between segments; where the number of blocks is
    not a multiple of four, FusedMM and SPMM keep the plain partition and SDDMM deals single blocks): the three ops on a
    prepared table against the oracle, every element."""
    assert torch.cuda.is_available()
    from paper_2311_00368_b200 import binding as b
    dev = lambda x: torch.from_numpy(np.ascontiguousarray(x)).cuda()
    rng = np.random.default_rng(7)
    b.debug_force_partition(2)
    try:
        for _ in range(6):
            M, K = int(rng.integers(2000, 40000)), int(rng.choice([512, 640, 1024, 1536, 2048, 2500, 4096]))
            Kd, N = int(rng.choice([32, 64, 100, 128])), int(rng.choice([32, 64, 128, 200, 256]))
            dens, kind = float(rng.choice([0.02, 0.04, 0.06])), str(rng.choice(["uniform", "powerlaw"]))
            p = W.small_random(int(rng.integers(1 << 30)), M, K, dens, Kd, N, kind=kind)
            use_bf, null = bool(rng.integers(0, 2)), bool(rng.random() < 0.25)
            what = f"M={M} K={K} Kd={Kd} N={N} d={dens} {kind} bf16={use_bf} null={null}"
            A, B, D, dt, cvt = p.A, p.B, p.D, torch.float32, dev
            if use_bf:
                A, B, D = (torch.from_numpy(np.ascontiguousarray(x)).to(torch.bfloat16).float().numpy() for x in (A, B, D))
                dt, cvt = torch.bfloat16, (lambda x: dev(x).to(torch.bfloat16))
            rp, ci, v, dA, dB, dD = dev(p.row_ptr), dev(p.col_idx), dev(p.values), cvt(A), cvt(B), cvt(D)
            ws = torch.empty(max(max(b.workspace_bytes(o, M, K, Kd, N, p.nnz) for o in range(3)), 1 << 20), dtype=torch.uint8, device="cuda")
            b.prepare_pattern(rp, ci, K, ws)
            sv, hv = (None, None) if null else (v, p.values)
            got = {"spmm": b.spmm(rp, ci, v, dD, K=K, workspace=ws, algo=4, dtype=dt),
                   "sddmm": b.sddmm(rp, ci, sv, dA, dB, workspace=ws, algo=4, dtype=dt),
                   "fusedmm": b.fusedmm(rp, ci, sv, dA, dB, dD, workspace=ws, algo=4, dtype=dt)}
            assert b.device_status(ws) == 0, what
            ref = {"spmm": oracle.spmm(p.row_ptr, p.col_idx, p.values, D), "sddmm": oracle.sddmm(p.row_ptr, p.col_idx, hv, A, B),
                   "fusedmm": oracle.fusedmm(p.row_ptr, p.col_idx, hv, A, B, D)}
            for op, out in got.items():
                ok, ratio = oracle.within_tolerance(out.cpu().numpy(), *ref[op])
                assert ok, f"{op}: {what}: worst error / allowed = {ratio:.3g}"
    finally:
        b.debug_force_partition(0)
