"""Multi-process plumbing of the benchmark: one process per GPU, no data-path collective.

The convolution path shards over the batch: every rank runs the same layers on its own images, and
nothing is exchanged.  What the ranks do share is timing: a step's duration is the maximum over the
ranks, and the job's throughput is the work of all ranks divided by that.  These helpers hold that
arithmetic so that it can be tested on CPU processes (gloo) as well as on GPUs (nccl).
"""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def env_ranks() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) as torchrun exports them; (0, 0, 1) for a plain launch."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def max_over_ranks(value: float, device) -> float:
    """The largest of `value` over all ranks (the value itself without a process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(work_per_rank: float, world: int, ms_per_step: float) -> float:
    """Whole-job units per second: every rank does `work_per_rank` per step (weak scaling), a step
    lasts as long as its slowest rank."""
    return world * work_per_rank / (ms_per_step * 1e-3)


def shard_images(global_batch: int, world: int, rank: int) -> Tuple[int, int]:
    """[first, last) image of `rank` when a global batch is dealt out in contiguous, near-equal parts."""
    base, extra = divmod(global_batch, world)
    first = rank * base + min(rank, extra)
    return first, first + base + (1 if rank < extra else 0)
