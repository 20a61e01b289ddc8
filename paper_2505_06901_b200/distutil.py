"""Rank bookkeeping for bench.py: the hot path shards with no data-path collective (every block is
independent), so the only cross-rank step is taking the slowest rank's device time."""
from __future__ import annotations

import os


def rank_info():
    """(rank, world_size, local_rank) from the torchrun environment; (0, 1, 0) when run directly."""
    return int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("LOCAL_RANK", "0"))


def max_over_ranks(values, dist=None, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch

    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def aggregate_throughput(bytes_per_rank: float, seconds_this_rank: float, world: int, dist=None, device="cpu") -> float:
    """Whole-job rate: every rank processed bytes_per_rank; the job took as long as its slowest rank."""
    (slowest,) = max_over_ranks([seconds_this_rank], dist, device)
    return world * bytes_per_rank / slowest if slowest > 0 else 0.0
