"""Multi-GPU plumbing of the hot path: requests are independent, so a job is batch shards, one process
per GPU, head matrices replicated, and no collective on the data path.  What ranks exchange is
bookkeeping only: a barrier around the timed region, the slowest rank's time, the units all ranks
processed.  Every function works on CPU tensors with the gloo backend and on CUDA tensors with nccl.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def world():
    """(rank, world_size) of the initialised process group, (0, 1) without one."""
    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(), dist.get_world_size()
    return 0, 1


def shard_seed(base_seed: int, rank: int) -> int:
    """Seed of a rank's synthetic shard: distinct per rank, the same for a rank on every run."""
    return int(base_seed) + 1000 * int(rank)


def shard_requests(n_requests: int, rank: int, world_size: int) -> range:
    """Contiguous slice of a batch of independent requests that a rank serves: every request lands on
    exactly one rank and slice sizes differ by at most one."""
    if not (0 <= rank < world_size):
        raise ValueError("rank outside the world")
    q, r = divmod(int(n_requests), int(world_size))
    lo = rank * q + min(rank, r)
    return range(lo, lo + q + (1 if rank < r else 0))


def _reduce(value: float, op, device) -> float:
    rank, n = world()
    if n == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=op)
    return float(t[0])


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's figure (device times are reported as the maximum over ranks)."""
    return _reduce(value, dist.ReduceOp.MAX, device)


def sum_over_ranks(value: float, device="cpu") -> float:
    return _reduce(value, dist.ReduceOp.SUM, device)


def job_throughput(units_this_rank: float, ms_this_rank: float, device="cpu"):
    """Whole-job throughput: the units all ranks processed over the slowest rank's time.
    Returns (units per second, that time in ms)."""
    ms = max_over_ranks(ms_this_rank, device)
    units = sum_over_ranks(units_this_rank, device)
    return units / (ms * 1e-3), ms
