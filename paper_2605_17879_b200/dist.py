"""Multi-process plumbing for the benchmark.

The scoring path does not shard across GPUs (a cross-rank median needs every rank of a
step on one device), so N GPUs run N independent replicas of the workload: no data-path
collective exists.  The only communication is the benchmark's own barrier and the
max-over-ranks reduction of the measured time.
"""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def env_world() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the launcher's environment (1 process if unset)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str) -> Tuple[int, int, int]:
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29533")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time: what a job of independent replicas waits for."""
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


def aggregate_throughput(units_this_rank: float, seconds_this_rank: float, device="cpu") -> Tuple[float, float]:
    """Whole-job throughput of independent replicas: units of all ranks / slowest rank's time.
    Returns (units_per_second, max_seconds)."""
    total = sum_over_ranks(units_this_rank, device)
    tmax = max_over_ranks(seconds_this_rank, device)
    return total / tmax, tmax


def finish() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
