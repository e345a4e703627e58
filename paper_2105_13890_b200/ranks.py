"""Host-side plumbing for runs with one process per GPU: rendezvous, barrier, max-over-ranks timing, aggregation,
and the all-reduce hook of data-parallel replicas.

By default every rank runs the whole per-GPU workload (replicas with no data-path collective); the only exchange
is the reduction of the ranks' timings, so that a whole-job number uses the slowest rank.  `reduce_hook` gives the
library's handles the all-reduce that makes replicas holding shares of one batch bit-identical to a single device
(integer maxima of the scale quantizers, integer sums of the gradients: both independent of reduction order).
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


class _DeviceBuffer:
    """A raw device pointer dressed as an array, so that torch can wrap it without copying."""

    def __init__(self, ptr: int, count: int, typestr: str):
        self.__cuda_array_interface__ = {"shape": (count,), "typestr": typestr, "data": (ptr, False), "version": 2, "strides": None}


def device_tensor(ptr: int, count: int, dtype_code: int) -> torch.Tensor:
    """The `count` int32 (code 0) or int64 (code 1) elements at device address `ptr`, as a tensor view."""
    return torch.as_tensor(_DeviceBuffer(ptr, count, "<i4" if dtype_code == 0 else "<i8"), device="cuda")


def reduce_hook(group=None):
    """An eoq.REDUCE_FN that all-reduces the buffer over the process group (MAX or SUM, in place, on the stream the
    library names).  Keep the returned object alive as long as a handle uses it."""
    from . import eoq

    def fn(user, ptr, count, dtype, op, stream):
        t = device_tensor(ptr, count, dtype)
        rop = dist.ReduceOp.MAX if op == eoq.EOQ_REDUCE_MAX else dist.ReduceOp.SUM
        if stream:
            with torch.cuda.stream(torch.cuda.ExternalStream(stream)):
                dist.all_reduce(t, op=rop, group=group)
        else:
            dist.all_reduce(t, op=rop, group=group)

    return eoq.REDUCE_FN(fn)


def finish() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
