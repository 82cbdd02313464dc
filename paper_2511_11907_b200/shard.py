"""Host-side logic of the multi-GPU run: the path shards by sequence with no data-path
collective, so every rank owns `batch` sequences of its own (weak scaling) and the only
communication is the barrier and the max-over-ranks of the timed region."""
from __future__ import annotations

import torch
import torch.distributed as dist


def rank_seed_offset(rank: int) -> int:
    """Distinct synthetic sequences per rank."""
    return int(rank)


def sequences_of_rank(batch_per_rank: int, rank: int):
    """Global sequence ids owned by `rank` (rank-major, contiguous)."""
    return range(rank * batch_per_rank, (rank + 1) * batch_per_rank)


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def aggregate_throughput(units_per_rank_per_step: float, steps: int, elapsed_ms_max: float, world: int) -> float:
    """Whole-job units/s: every rank processed the same number of units; time is the slowest rank's."""
    return world * units_per_rank_per_step * steps / (elapsed_ms_max * 1e-3)
