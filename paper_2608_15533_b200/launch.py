"""One process per GPU: rendezvous, row sharding and max-over-ranks timing.

The decode path has no exchange step -- every (sequence, head) unit owns its base, its log and its
metadata and never reads another unit's -- so ranks split the batch rows and run independently.
``torch.distributed`` is used only for the barrier around the timed region and for taking the
maximum of the per-rank durations; there is no data-path collective.
"""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def world() -> Tuple[int, int, int]:
    """(rank, world_size, local_rank) from the launcher's environment (1 process if unset)."""
    return (int(os.environ.get("RANK", 0)), int(os.environ.get("WORLD_SIZE", 1)),
            int(os.environ.get("LOCAL_RANK", 0)))


def init(backend: str = "nccl") -> Tuple[int, int, int]:
    """Join the process group when launched with more than one rank; returns ``world()``."""
    rank, size, local = world()
    if size > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        if backend == "nccl":
            torch.cuda.set_device(local)
            dist.init_process_group(backend, device_id=torch.device("cuda", local))
        else:
            dist.init_process_group(backend)
    return rank, size, local


def shard_rows(global_rows: int, world_size: int, rank: int) -> Tuple[int, int]:
    """Contiguous block of batch rows owned by ``rank``: ``(first_row, n_rows)``; remainders go to
    the lowest ranks so that block sizes differ by at most one."""
    base, extra = divmod(global_rows, world_size)
    n = base + (1 if rank < extra else 0)
    first = rank * base + min(rank, extra)
    return first, n


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device=None) -> float:
    """Maximum of a per-rank scalar (device-timed milliseconds) over all ranks."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device=None) -> float:
    """Sum of a per-rank scalar (units processed) over all ranks."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def finalize() -> None:
    if dist.is_initialized():
        dist.barrier()
        dist.destroy_process_group()
