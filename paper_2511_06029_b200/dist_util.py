"""Multi-rank plumbing of the benchmark: one process per GPU, sequences sharded across ranks, no collective on
the data path.  The only exchanges are the barrier around the timed region and the reduction of each rank's
(elapsed time, units processed) into the whole-job figure: max of the times, sum of the units."""
from __future__ import annotations

from typing import Sequence, Tuple

import torch


def rank_batch_ids(rank: int, per_rank_batch: int) -> torch.Tensor:
    """Global sequence ids owned by `rank` (weak scaling: every rank holds `per_rank_batch` sequences)."""
    return torch.arange(rank * per_rank_batch, (rank + 1) * per_rank_batch)


def reduce_job(dist, device, times_ms: Sequence[float], units: Sequence[float]) -> Tuple[list, list]:
    """Max over ranks of each time and sum over ranks of each unit count (identity when dist is None)."""
    if dist is None:
        return list(times_ms), list(units)
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    u = torch.tensor(list(units), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return t.tolist(), u.tolist()


def job_value(units_total: float, max_time_ms: float) -> float:
    """Whole-job throughput: all units of all ranks over the slowest rank's time."""
    return units_total / (max_time_ms * 1e-3)
