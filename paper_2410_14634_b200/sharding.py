"""Host-side plumbing for running the layer on several GPUs (one process per GPU).

Images are independent in x = f^{-1}(y), grad_y and f, so the batch is split
across ranks with no exchange on the data path.  Only grad_w is a sum over the
batch (Theorem 2 sums over pixels, Algorithm 1 over the batch): in data-parallel
training each rank's grad_w is summed with one all-reduce of C*C*k*k floats.
`torch.distributed` is used as is (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist


def shard_batch(B: int, world: int, rank: int) -> Tuple[int, int]:
    """(start, count) of the images rank `rank` of `world` owns; counts differ by at most one."""
    if world < 1 or not (0 <= rank < world):
        raise ValueError("bad world/rank")
    base, extra = divmod(B, world)
    start = rank * base + min(rank, extra)
    return start, base + (1 if rank < extra else 0)


def allreduce_grad_w(grad_w: torch.Tensor) -> torch.Tensor:
    """Sum per-rank weight gradients in place over the default process group."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(grad_w, op=dist.ReduceOp.SUM)
    return grad_w


def max_over_ranks(value: float, device=None) -> float:
    """The maximum of a per-rank scalar (device time of a step) over all ranks."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
