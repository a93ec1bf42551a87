"""Host logic of the multi-GPU path on CPU: two gloo ranks, problem assignment and the
max/sum reductions that turn per-rank timings into one whole-job number."""
import os
import socket

import torch.multiprocessing as mp

from paper_2311_00368_b200 import replicas


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    r, lr, w = replicas.init("gloo")
    assert (r, lr, w) == (rank, rank, world)
    replicas.barrier()
    t_max = replicas.max_over_ranks(1.0 + rank)
    f_sum = replicas.sum_over_ranks(10.0 * (rank + 1))
    out.put((rank, t_max, f_sum, replicas.assign_problems(8, rank, world),
             replicas.instance_seed(4, rank)))


def test_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [2.0, 2.0]      # max over ranks
    assert [r[2] for r in res] == [30.0, 30.0]    # sum over ranks
    assert res[0][3] == [0, 2, 4, 6] and res[1][3] == [1, 3, 5, 7]
    assert res[0][4] == 4 and res[1][4] == 1004


def test_single_process_defaults(monkeypatch):
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        monkeypatch.delenv(k, raising=False)
    assert replicas.env_world() == (0, 0, 1)
    assert replicas.max_over_ranks(3.5) == 3.5 and replicas.sum_over_ranks(2.0) == 2.0
    assert replicas.assign_problems(8, 0, 1) == list(range(8))


def _shard_worker(rank, world, port, out):
    """One rank of a row-sharded run on CPU: its slice of S, the oracle on the slice, results gathered."""
    import numpy as np
    import torch
    import torch.distributed as dist
    import oracle
    from paper_2311_00368_b200 import workloads as W
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    replicas.init("gloo")
    p = W.small_random(9000, 301, 400, 0.2, 16, 24, kind="powerlaw")
    r0, r1, rp, ci, v, A = replicas.row_shard(p.row_ptr, p.col_idx, p.values, rank, world, A=p.A)
    O_loc, _ = oracle.fusedmm(rp, ci, v, A, p.B, p.D)          # B and D are replicated
    C_loc, _ = oracle.sddmm(rp, ci, v, A, p.B)
    # gather the shards' outputs on every rank (sizes differ: pad to the largest)
    sizes = [torch.zeros(2, dtype=torch.int64) for _ in range(world)]
    dist.all_gather(sizes, torch.tensor([r1 - r0, len(ci)]))
    rows_max, nnz_max = int(max(s[0] for s in sizes)), int(max(s[1] for s in sizes))
    buf = torch.zeros(rows_max * p.N + nnz_max, dtype=torch.float64)
    buf[:(r1 - r0) * p.N] = torch.from_numpy(O_loc.reshape(-1))
    buf[rows_max * p.N:rows_max * p.N + len(ci)] = torch.from_numpy(C_loc)
    bufs = [torch.zeros_like(buf) for _ in range(world)]
    dist.all_gather(bufs, buf)
    O = np.concatenate([bufs[r][:int(sizes[r][0]) * p.N].numpy().reshape(-1, p.N) for r in range(world)])
    C = np.concatenate([bufs[r][rows_max * p.N:rows_max * p.N + int(sizes[r][1])].numpy() for r in range(world)])
    O_ref, _ = oracle.fusedmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D)
    C_ref, _ = oracle.sddmm(p.row_ptr, p.col_idx, p.values, p.A, p.B)
    out.put((rank, bool(np.array_equal(O, O_ref)), bool(np.array_equal(C, C_ref)), r0, r1, len(ci)))


def test_row_shards_of_two_gloo_ranks_reassemble_the_whole_problem():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_shard_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert all(r[1] and r[2] for r in res), "concatenated shard outputs differ from the whole problem's"
    assert res[0][3] == 0 and res[0][4] == res[1][3] and res[1][4] == 301      # contiguous, complete
    total = res[0][5] + res[1][5]
    assert abs(res[0][5] - total / 2) < 0.05 * total                            # balanced by stored entries


def test_row_shard_bounds_edge_cases():
    import numpy as np
    assert replicas.row_shard_bounds(np.array([0, 0, 0, 0]), 2) == [0, 0, 3]            # no entries at all
    assert replicas.row_shard_bounds(np.array([0, 10]), 4) == [0, 1, 1, 1, 1]            # one row, four ranks
    b = replicas.row_shard_bounds(np.arange(0, 101, 10), 1)
    assert b == [0, 10]
    rp = np.array([0, 5, 5, 5, 20, 40])
    b = replicas.row_shard_bounds(rp, 2)
    assert b[0] == 0 and b[-1] == 5 and b == sorted(b)
    r0, r1, rp1, ci, v, A = replicas.row_shard(rp, np.arange(40), np.arange(40.0), 1, 2, A=np.arange(10).reshape(5, 2))
    assert rp1[0] == 0 and rp1[-1] == len(ci) == len(v) and len(A) == r1 - r0
