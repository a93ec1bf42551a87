"""Multi-GPU plumbing: independent replicas or row shards, no data-path collective.

The three ops are row-independent (Alg. 1-3 work on one row of S at a time) and every benchmark
problem is an independent instance.  A multi-GPU run therefore either gives each rank its own
instance (weak scaling) or cuts ONE problem into contiguous row ranges of about equal stored entries
(`row_shard`, strong scaling: a rank holds its rows of S, A and O and all of B and D); either way only
the *timing* is reduced across ranks (max), through torch.distributed.  Works with the nccl backend on
GPUs and with gloo on CPU (used by the tests).  This module only slices arrays; it holds none of the
ops' arithmetic.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world():
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) when absent."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def instance_seed(base_seed: int, rank: int) -> int:
    """Seed of the problem instance a rank works on: rank 0 keeps the named workload's seed."""
    return base_seed + 1000 * rank


def assign_problems(num_problems: int, rank: int, world_size: int) -> list:
    """Round-robin assignment of independent problems (e.g. batch x heads) to ranks."""
    return list(range(rank, num_problems, world_size))


def row_shard_bounds(row_ptr, world_size: int) -> list:
    """Row boundaries [r_0 = 0, r_1, ..., r_world = M] of a 1-D partition of S into contiguous row ranges
    with about nnz / world_size stored entries each (rows are never split; empty shards are possible)."""
    import numpy as np
    row_ptr = np.asarray(row_ptr)
    M, nnz = len(row_ptr) - 1, int(row_ptr[-1])
    targets = [nnz * r // world_size for r in range(1, world_size)]
    cuts = [int(np.searchsorted(row_ptr, t, side="left")) for t in targets]
    bounds = [0] + [min(max(c, 0), M) for c in cuts] + [M]
    for i in range(1, len(bounds)):          # monotone
        bounds[i] = max(bounds[i], bounds[i - 1])
    return bounds


def row_shard(row_ptr, col_idx, values, rank: int, world_size: int, A=None):
    """The rank's share of a CSR matrix (and of the row-aligned dense operand A): (r0, r1, row_ptr re-based to
    0, col_idx slice, values slice, A rows).  Outputs of the shard are rows r0..r1 of O (SPMM / FusedMM) or the
    entries row_ptr[r0]..row_ptr[r1] of the SDDMM result; concatenating the ranks' outputs gives the whole."""
    import numpy as np
    b = row_shard_bounds(row_ptr, world_size)
    r0, r1 = b[rank], b[rank + 1]
    p0, p1 = int(row_ptr[r0]), int(row_ptr[r1])
    rp = (np.asarray(row_ptr[r0:r1 + 1]) - p0).astype(np.int32)
    return r0, r1, rp, col_idx[p0:p1], values[p0:p1], (None if A is None else A[r0:r1])


def init(backend: str, device=None):
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        kw = {}
        if device is not None and backend == "nccl":
            kw["device_id"] = device
        dist.init_process_group(backend=backend, **kw)
    return rank, local_rank, world


def barrier():
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
