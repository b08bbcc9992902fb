"""Host-side logic of multi-GPU runs: the path partitions over independent sequences (each has its own
scores, thresholds and masks), so ranks share nothing on the data path.  What is left is bookkeeping:
which sequences a rank owns, and the whole-job rate = all ranks' units / the slowest rank's time."""
from __future__ import annotations

from typing import List, Tuple

import torch
import torch.distributed as dist


def shard_range(n_units: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous, balanced [lo, hi) of n_units for this rank (sizes differ by at most one)."""
    if not (0 <= rank < world):
        raise ValueError("rank outside [0, world)")
    return (n_units * rank) // world, (n_units * (rank + 1)) // world


def shard_sizes(n_units: int, world: int) -> List[int]:
    return [shard_range(n_units, r, world)[1] - shard_range(n_units, r, world)[0] for r in range(world)]


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time (or any per-rank scalar's maximum); identity without a process group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_rate(units_this_rank: float, elapsed_ms_this_rank: float, device="cpu") -> Tuple[float, float]:
    """(units of all ranks per second, the slowest rank's milliseconds)."""
    ms = max_over_ranks(elapsed_ms_this_rank, device)
    units = sum_over_ranks(units_this_rank, device)
    return units / (ms * 1e-3), ms
