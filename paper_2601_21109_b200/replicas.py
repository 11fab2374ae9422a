"""Multi-GPU plumbing of the benchmark: independent replicas, one process per GPU.

The hot path has no exchange step (sequences and rows are independent in all three calls), so N GPUs
run N replicas with no collective on the data path.  What the ranks share is only the timing protocol:
a barrier on both sides of the timed region and the MAX over ranks of its device-timed duration; the
job's throughput is the units all ranks processed over that time (weak scaling)."""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def world_from_env() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) as torch.distributed.run exports them; (0, 0, 1) without it."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str, local_rank: int, world: int) -> None:
    """Joins the process group when there is more than one rank (nccl on GPUs, gloo on CPU)."""
    if world <= 1 or dist.is_initialized():
        return
    if backend == "nccl":
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    else:
        dist.init_process_group(backend)


def barrier(world: int, cuda: bool = True) -> None:
    if world > 1:
        dist.barrier()
    if cuda:
        torch.cuda.synchronize()


def max_over_ranks(value: float, world: int, device: str = "cuda") -> float:
    """The slowest rank's figure: a multi-GPU time is the max over ranks, never one rank's own."""
    if world <= 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank_per_step: int, steps: int, world: int, ms_max: float) -> float:
    """Whole-job units per second: every rank processed its own units in the slowest rank's time."""
    return units_per_rank_per_step * steps * world / (ms_max * 1e-3)


def finish(world: int) -> None:
    if world > 1 and dist.is_initialized():
        dist.destroy_process_group()
