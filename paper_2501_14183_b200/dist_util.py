"""Multi-GPU plumbing of the benchmark: the path shards over batches (every rank hashes, selects and attends on its
own batch, exactly the per-batch method of the paper), so there is no data-path collective; ranks only agree on the
slowest time."""
from __future__ import annotations

import torch


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of the synthetic batch of `rank`: every rank gets different data of the same shape."""
    return base_seed + 1000 * rank


def max_over_ranks(values, dist=None, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def aggregate_throughput(units_per_rank: int, world: int, max_seconds: float) -> float:
    """Whole-job throughput under weak scaling: all ranks' units over the slowest rank's time."""
    return units_per_rank * world / max_seconds
