"""Data-parallel plumbing: one process per GPU, every rank evicts its own requests.

The eviction of one request never reads another request's cache (Algorithm 1 works per
sequence; Algorithm 2 shares a budget only across the layers of one sequence), so ranks
exchange no cache data.  What crosses ranks is bookkeeping only: which requests a rank serves,
the slowest rank's time and the number of tokens all ranks processed.
"""
from __future__ import annotations

from typing import Sequence

import torch
import torch.distributed as dist


def shard_requests(n_requests: int, rank: int, world: int) -> range:
    """Contiguous, balanced split: the first ``n_requests % world`` ranks get one extra."""
    if not (0 <= rank < world):
        raise ValueError("rank %d outside world of %d" % (rank, world))
    base, extra = divmod(int(n_requests), int(world))
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def _device_for_group() -> torch.device:
    # NCCL reduces device tensors; gloo reduces host tensors
    if dist.get_backend() == "nccl":
        return torch.device("cuda", torch.cuda.current_device())
    return torch.device("cpu")


def slowest_rank_ms(ms: float) -> float:
    """MAX over ranks of a device-measured duration (the whole job ends with its slowest rank)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([float(ms)], dtype=torch.float64, device=_device_for_group())
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_units(units_this_rank: int) -> int:
    """SUM over ranks of the units (tokens) each rank processed."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return int(units_this_rank)
    t = torch.tensor([int(units_this_rank)], dtype=torch.int64, device=_device_for_group())
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return int(t.item())


def whole_job_throughput(units_this_rank: int, ms_this_rank: float) -> float:
    """Units of all ranks divided by the slowest rank's time, in units per second."""
    ms = slowest_rank_ms(ms_this_rank)
    return whole_job_units(units_this_rank) / (ms * 1e-3)
