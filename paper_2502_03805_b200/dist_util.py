"""Multi-rank bookkeeping for the benchmark: which layers a rank owns and the max-over-ranks time.

The compression of one layer is independent of every other layer, so ranks share nothing on the data path; the only
exchanges are a barrier and one MAX all-reduce of the measured time.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def rank_layer_ids(rank: int, layers_per_rank: int):
    """Seeds of the layers rank `rank` generates: disjoint across ranks, `layers_per_rank` each (weak scaling)."""
    return list(range(rank * layers_per_rank, (rank + 1) * layers_per_rank))


def max_over_ranks(value: float, device=None) -> float:
    """MAX all-reduce of a host scalar (identity when torch.distributed is not initialised)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(units_per_rank: int, world: int, seconds_max: float) -> float:
    """Units processed by all ranks divided by the slowest rank's time."""
    return units_per_rank * world / seconds_max
