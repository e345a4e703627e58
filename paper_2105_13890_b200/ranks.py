"""Host-side plumbing for runs with one process per GPU: rendezvous, barrier, max-over-ranks timing, aggregation.

The path has no data-path collective (replicas only: every rank runs the whole per-GPU workload); the only
exchange is the reduction of the ranks' timings, so that a whole-job number uses the slowest rank.
Works with the NCCL backend on GPUs and with gloo on CPU (tests).
"""
from __future__ import annotations

import os
from typing import Sequence

import torch
import torch.distributed as dist


def world() -> tuple[int, int, int]:
    """(world size, rank, local rank) from the launcher's environment; (1, 0, 0) for a plain `python` run."""
    return int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0"))


def init(backend: str, device: torch.device | None = None) -> None:
    if world()[0] > 1 and not dist.is_initialized():
        if backend == "nccl" and device is not None:
            dist.init_process_group(backend, device_id=device)
        else:
            dist.init_process_group(backend)


def barrier(sync_cuda: bool = True) -> None:
    if dist.is_initialized():
        dist.barrier()
    if sync_cuda and torch.cuda.is_available():
        torch.cuda.synchronize()


def max_over_ranks(values: Sequence[float], device: str | torch.device = "cpu") -> list[float]:
    """Element-wise maximum of each rank's list of timings."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_initialized():
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_rate(units_per_rank_step: float, steps: int, slowest_ms: float, world_size: int) -> float:
    """Units per second of the whole job: every rank did `steps` steps of `units_per_rank_step` in `slowest_ms`."""
    return world_size * units_per_rank_step * steps / (slowest_ms / 1e3)


def finish() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
