"""Multi-GPU plumbing for the benchmark: independent replicas, one process per GPU.

The linear layer of a single-user draft model does not shard: every GPU would need the whole
activation vector and would own a slice of a microsecond-long kernel.  So N GPUs run N
independent replicas of the same workload (weak scaling, no collective on the data path).
torch.distributed is used only to line the replicas up and to combine their timings.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world():
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) outside it."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str) -> None:
    """Join the process group if the environment describes more than one rank."""
    if env_world()[2] > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend=backend)


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest replica's time: what a whole-job throughput must be computed from."""
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


def whole_job_throughput(units_per_rank: float, seconds_this_rank: float, device="cpu") -> float:
    """Units processed by all replicas divided by the slowest replica's time."""
    total = sum_over_ranks(units_per_rank, device)
    slowest = max_over_ranks(seconds_this_rank, device)
    return total / slowest


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
