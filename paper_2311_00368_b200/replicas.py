"""Multi-GPU plumbing: independent replicas, no data-path collective.

The three ops are row-independent and every benchmark problem is an independent instance, so a
multi-GPU run gives each rank its own instance (weak scaling) and only the *timing* is reduced
across ranks (max), through torch.distributed.  Works with the nccl backend on GPUs and with
gloo on CPU (used by the tests).
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
