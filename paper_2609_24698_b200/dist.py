"""Process-group plumbing for multi-GPU runs.

The verify path does not exchange data between sequences, so N GPUs run N independent
replicas of the workload (no data-path collective).  The only communication is for
measurement: a barrier on both sides of the timed region and a MAX over ranks of the
device time.  Works with `nccl` on GPUs and `gloo` on CPU (tests).
"""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def env_world() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) outside it."""
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def init(backend: str) -> Tuple[int, int]:
    rank, _, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(x: float, device="cpu") -> float:
    if not dist.is_initialized():
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float, device="cpu") -> float:
    if not dist.is_initialized():
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_throughput(units_local: float, seconds_local: float, device="cpu") -> Tuple[float, float]:
    """(units of all ranks / max time over ranks, that max time)."""
    t = max_over_ranks(seconds_local, device)
    u = sum_over_ranks(units_local, device)
    return u / t, t


def finalize() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
