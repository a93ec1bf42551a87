"""b2sp_spmm_static_scratch -- the entry point for callers that cannot allocate device memory
(a plug-in living inside a host process that owns the whole device-memory arena, or a loop that
may not trigger an allocation's synchronisation).  Its scratch is a fixed array inside the library.

The file name makes pytest collect it last, so that with `-x` every other test has already run.
It checks, through the C ABI, that two calls in a row (the second on a different, smaller problem,
so anything the first call left in the shared scratch is stale) give what the regular entry point
gives, within the tolerance the parity tests use, and that the size limit is enforced.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2311_00368_b200 import workloads as W

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-5, 1e-6


def _dev(x):
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def test_static_scratch_matches_regular_entry_point_twice_in_a_row():
    assert torch.cuda.is_available()
    from paper_2311_00368_b200 import binding as b

    problems = [W.small_random(301, 700, 512, 0.2, 0, 128, kind="powerlaw"),
                W.small_random(302, 90, 300, 0.3, 0, 64)]
    staged = []
    for p in problems:
        rp, ci, v, D = map(_dev, (p.row_ptr, p.col_idx, p.values, p.D))
        want = b.spmm(rp, ci, v, D, algo=b.ALGO_ROW)
        out = torch.full((p.M, p.N), float("nan"), device="cuda")
        staged.append((p, rp, ci, v, D, want, out))
    torch.cuda.synchronize()
    # two calls back to back on one stream, no synchronisation in between
    for p, rp, ci, v, D, want, out in staged:
        b.spmm_static_scratch(rp, ci, v, D, out=out)
    torch.cuda.synchronize()
    for p, rp, ci, v, D, want, out in staged:
        _, T = oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D)
        ok, ratio = oracle.within_tolerance(out.cpu().numpy(), want.cpu().numpy().astype(np.float64),
                                            T, RTOL, ATOL)
        assert ok, f"static-scratch SPMM differs from b2sp_spmm by {ratio:.3g} x the tolerance"
        ref, _ = oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D)
        ok, ratio = oracle.within_tolerance(out.cpu().numpy(), ref, T, RTOL, ATOL)
        assert ok, f"static-scratch SPMM differs from the oracle by {ratio:.3g} x the tolerance"


def test_static_scratch_rejects_oversized_problems():
    from paper_2311_00368_b200 import binding as b
    M = b.STATIC_SCRATCH_MAX_ROWS + 1
    rp = torch.zeros(M + 1, dtype=torch.int32, device="cuda")
    e_i = torch.zeros(0, dtype=torch.int32, device="cuda")
    e_f = torch.zeros(0, dtype=torch.float32, device="cuda")
    D = torch.zeros((4, 4), dtype=torch.float32, device="cuda")
    with pytest.raises(b.B2spError) as e:
        b.spmm_static_scratch(rp, e_i, e_f, D)
    assert e.value.status == 7
    assert "scratch" in str(e.value)


def test_static_scratch_takes_the_largest_problem_it_promises():
    """M equal to the limit is the one size at which the built-in array is exactly as large as the
    workspace the regular entry point would ask for; most rows are empty, a few carry entries."""
    from paper_2311_00368_b200 import binding as b
    M, K, N = b.STATIC_SCRATCH_MAX_ROWS, 64, 32
    rng = np.random.default_rng(11)
    lens = np.zeros(M, dtype=np.int64)
    busy = rng.choice(M, size=500, replace=False)
    lens[busy] = rng.integers(1, K + 1, size=busy.size)
    lens[M - 1] = K                       # the last row too
    row_ptr = np.zeros(M + 1, dtype=np.int32)
    row_ptr[1:] = np.cumsum(lens)
    col_idx = np.concatenate([np.sort(rng.choice(K, size=l, replace=False)) for l in lens[lens > 0]]).astype(np.int32)
    values = W.values_uniform(rng, int(row_ptr[-1]))
    D = W.dense_normal(rng, K, N)
    out = torch.full((M, N), float("nan"), device="cuda")
    b.spmm_static_scratch(_dev(row_ptr), _dev(col_idx), _dev(values), _dev(D), K=K, out=out)   # B2SP_OK or it raises
    ref, T = oracle.spmm(row_ptr, col_idx, values, D)
    ok, ratio = oracle.within_tolerance(out.cpu().numpy(), ref, T, RTOL, ATOL)
    assert ok, f"static-scratch SPMM at the size limit differs from the oracle by {ratio:.3g} x the tolerance"
