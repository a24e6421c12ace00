"""World-size-2 checks of the benchmark's multi-rank plumbing on CPU (gloo): sequence sharding is disjoint and
complete, the job figure is sum(units) / max(time), and ranks see different synthetic sequences."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2511_06029_b200 import dist_util, synth


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close(); return p


def _worker(rank, world, port, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"; os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ids = dist_util.rank_batch_ids(rank, 4)
        gathered = [torch.zeros(4, dtype=torch.int64) for _ in range(world)]
        dist.all_gather(gathered, ids)
        # each rank "measures" a different time and unit count
        times, units = dist_util.reduce_job(dist, torch.device("cpu"), [10.0 + 5 * rank, 3.0 - rank], [100.0 * (rank + 1), 7.0])
        w = synth.shrink(synth.WORKLOADS["llama8b"], n_layers=1, batch=8)
        fl = synth.anchor_flags(w, torch.arange(64), ids)
        ret[rank] = (torch.cat(gathered).tolist(), times, units, fl.sum().item(), fl.shape)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_rank_sharding_and_reduction():
    world = 2
    mgr = mp.Manager(); ret = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), ret), nprocs=world, join=True)
    for rank in range(world):
        all_ids, times, units, _, shape = ret[rank]
        assert all_ids == list(range(8))                      # disjoint and complete
        assert times == [15.0, 3.0] and units == [300.0, 14.0]  # max of times, sum of units, same on every rank
        assert tuple(shape) == (1, 4, 64)
    assert dist_util.job_value(300.0, 15.0) == 20000.0
    t, u = dist_util.reduce_job(None, None, [1.0], [2.0])
    assert t == [1.0] and u == [2.0]
