"""Host-side helpers for running independent replicas, one process per GPU.

The path has no exchange step: gradient elements are owned by exactly one thread, so several GPUs
run independent replicas and nothing crosses NVLink.  What the processes share is only the timing
protocol of the benchmark: a barrier on both sides of the timed region and the maximum over ranks
of the device time.
"""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def rank_info() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the launcher's environment (1 process if absent)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str) -> bool:
    """Joins the process group when launched with more than one rank; returns True if distributed."""
    _, _, world = rank_info()
    if world <= 1:
        return False
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29512")
    dist.init_process_group(backend)
    return True


def barrier(distributed: bool) -> None:
    if distributed:
        dist.barrier()
    if torch.cuda.is_available():
        torch.cuda.synchronize()


def max_over_ranks(value: float, distributed: bool, device: torch.device) -> float:
    """The slowest rank defines the time of a step."""
    if not distributed:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, seconds: float, world: int) -> float:
    """Whole-job throughput of `world` replicas that each processed units_per_rank in `seconds`."""
    return world * units_per_rank / seconds


def finish(distributed: bool) -> None:
    if distributed:
        dist.barrier()
        dist.destroy_process_group()
