"""Multi-rank plumbing of the benchmark: one process per GPU, sequences sharded across ranks, no collective on
the data path.  The only exchanges are the barrier around the timed region and the reduction of each rank's
(elapsed time, units processed) into the whole-job figure: max of the times, sum of the units."""
from __future__ import annotations

import os
import socket
import subprocess
from typing import Sequence, Tuple

import torch


def spawn_ranks(cmd: Sequence[str], n: int, timeout_s: float = 3600.0) -> int:
    """Start `cmd` n times as the ranks of one job on this node (what a launcher would do): RANK / LOCAL_RANK =
    0..n-1, WORLD_SIZE = n, rendezvous on 127.0.0.1 at a free port.  The ranks inherit stdout / stderr, so rank
    0's result line reaches the caller's stdout.  Returns 0 if every rank exited 0; otherwise the remaining ranks
    are stopped (by their own pids) and the first non-zero exit code is returned."""
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), LOCAL_WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen(list(cmd), env=env))
    import time
    deadline = time.monotonic() + timeout_s
    rc = 0
    pending = set(range(n))
    while pending and rc == 0:
        for r in sorted(pending):
            code = procs[r].poll()
            if code is not None:
                pending.discard(r)
                if code != 0:
                    rc = code
        if time.monotonic() > deadline:
            rc = 124
        if pending and rc == 0:
            time.sleep(0.05)
    for r in pending:                                    # a rank failed or the job ran out of time: stop the others
        procs[r].terminate()
    for r in pending:
        try:
            procs[r].wait(timeout=10)
        except subprocess.TimeoutExpired:
            procs[r].kill()
    return rc


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


def allreduce_layer_sparsity(dist, local_sparsity: torch.Tensor, local_kv_heads: int, total_kv_heads: int) -> torch.Tensor:
    """Layer sparsity of a cache sharded by KV head (tensor-parallel attention).

    `lethe_estimate_sparsity` returns, per (layer, sequence), the mean Hoyer sparsity over the KV heads a rank
    holds.  The layer value of Sec. 4.2 is the mean over all heads, so ranks exchange one [L][B] fp32 tensor per
    prune round: sum over ranks of (local mean x local head count), divided by the total head count.  Every rank
    then calls `lethe_alloc_budgets` on the same values and, the allocator being integer arithmetic, gets the
    same budgets.  This is the only exchange a head-sharded run of the path needs.
    """
    s = local_sparsity.to(torch.float32) * float(local_kv_heads)
    if dist is not None:
        dist.all_reduce(s, op=dist.ReduceOp.SUM)
    return s / float(total_kv_heads)
