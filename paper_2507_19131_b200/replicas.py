"""Multi-GPU plumbing of the benchmark: the path shards by image (images are independent and the window selection is
per image), so N GPUs run N replicas with no data-path collective.  What is shared is only the bookkeeping below:
which input a rank works on, the max-over-ranks device time, and the whole-job throughput.  Works on any
torch.distributed backend (NCCL on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

import numpy as np
import torch
import torch.distributed as dist


def rank_input(x: np.ndarray, rank: int) -> np.ndarray:
    """The image a rank processes: the seeded workload, cyclically shifted along the rows by the rank, so that
    replicas do not compute identical data (weak scaling: one image per rank per step)."""
    return np.ascontiguousarray(np.roll(x, rank, axis=1))


def max_over_ranks(ms: float, device="cpu") -> float:
    """Device time of the slowest rank (every multi-GPU number is the max over ranks)."""
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(images_per_rank_per_step: int, steps: int, world: int, max_ms: float) -> float:
    """Whole-job images/s: what all ranks processed divided by the slowest rank's time."""
    return world * images_per_rank_per_step * steps / (max_ms / 1e3)
