"""Host-side plumbing for running the path on several GPUs of one node.

The merge-layer step is independent per request (per-request softmax, top-k,
kept set and offsets), so it shards by request with no exchange step on the
data path: every rank runs the same kernels on its own requests.  The only
communication is a barrier around the timed region and a MAX reduction of the
per-rank device time.  Works with the ``nccl`` backend on GPUs and with
``gloo`` on CPU tensors (used by the tests).
"""
from __future__ import annotations

from typing import List, Sequence

import torch
import torch.distributed as dist


def world() -> int:
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def shard_requests(n_requests: int, rank: int, world_size: int) -> List[int]:
    """Request indices owned by ``rank``: contiguous blocks, sizes differing by at most one."""
    if world_size <= 0 or not (0 <= rank < world_size):
        raise ValueError("bad rank / world size")
    base, extra = divmod(n_requests, world_size)
    lo = rank * base + min(rank, extra)
    return list(range(lo, lo + base + (1 if rank < extra else 0)))


def max_over_ranks(value: float, device=None) -> float:
    """MAX of a per-rank scalar (the slowest rank's device time decides)."""
    if world() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device=None) -> float:
    if world() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_steps_per_second(steps_this_rank: Sequence[float], seconds_this_rank: float, device=None) -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    total = sum_over_ranks(float(sum(steps_this_rank)), device)
    return total / max_over_ranks(seconds_this_rank, device)
