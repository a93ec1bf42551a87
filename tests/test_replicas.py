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
