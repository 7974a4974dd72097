"""Host-side helpers of the benchmark: rank set-up and the max-over-ranks reduction.

The path does not shard: the layer of the paper runs on one GPU.  With N ranks every rank runs
its own replica on its own synthetic batch (weak scaling, no data-path collective); the only
communication is the barrier around the timed region and the reduction of the per-rank times.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def rank_info():
    """(rank, local_rank, world_size) from the launcher's environment (1 process if absent)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init_process_group(backend: str):
    """Join the launcher's rendezvous when there is more than one rank."""
    rank, _, world = rank_info()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world


def barrier():
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time: what a multi-GPU number is quoted on."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    """Units of work all ranks processed together."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_throughput(units_this_rank: float, seconds_this_rank: float, device="cpu") -> float:
    """(units of all ranks) / (time of the slowest rank)."""
    return sum_over_ranks(units_this_rank, device) / max_over_ranks(seconds_this_rank, device)
