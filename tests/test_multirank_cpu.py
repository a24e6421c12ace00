"""World-size-2 checks of the benchmark's multi-rank plumbing on CPU (gloo): sequence sharding is disjoint and
complete, the job figure is sum(units) / max(time), and ranks see different synthetic sequences."""
import json
import os
import socket
import subprocess
import sys

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


def _tp_worker(rank, world, port, ret):
    """Each rank holds half of the KV heads of the same cache; after the one all-reduce both must allocate the
    budgets an unsharded run allocates, and prune their own heads exactly as the unsharded run prunes them."""
    import oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"; os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        L, B, Hq, Hkv, D, cap, n = 4, 2, 8, 4, 8, 96, 80
        g = torch.Generator().manual_seed(5)
        k = torch.randn((L, B, Hkv, cap, D), generator=g); v = torch.randn((L, B, Hkv, cap, D), generator=g)
        rel = torch.rand((L, B, Hkv, cap), generator=g) ** 4
        pos = torch.arange(cap, dtype=torch.int32).expand(L, B, Hkv, cap).contiguous()
        full = oracle.OracleCache(L, B, Hq, Hkv, D, cap, k.clone(), v.clone(), rel.clone(), pos.clone(),
                                  torch.full((L, B, Hkv), n, dtype=torch.int32))
        hs = slice(rank * 2, rank * 2 + 2)
        mine = oracle.OracleCache(L, B, Hq // 2, 2, D, cap, k[:, :, hs].contiguous(), v[:, :, hs].contiguous(),
                                  rel[:, :, hs].contiguous(), pos[:, :, hs].contiguous(),
                                  torch.full((L, B, 2), n, dtype=torch.int32))
        T = torch.tensor([L * 40, L * 55], dtype=torch.int64)
        _, S_full = oracle.estimate_sparsity(full)
        _, bud_full = oracle.alloc_budgets(S_full, T, 12)
        oracle.rasr_prune(full, bud_full, 8, 4)
        _, S_loc = oracle.estimate_sparsity(mine)
        S_all = dist_util.allreduce_layer_sparsity(dist, S_loc, 2, Hkv)
        _, bud = oracle.alloc_budgets(S_all.contiguous(), T, 12)
        oracle.rasr_prune(mine, bud, 8, 4)
        ret[rank] = (torch.allclose(S_all, S_full, atol=1e-6), torch.equal(bud, bud_full),
                     torch.equal(mine.len, full.len[:, :, hs]), torch.equal(mine.pos, full.pos[:, :, hs]),
                     torch.equal(mine.k, full.k[:, :, hs]))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_rank_head_sharded_prune_round():
    mgr = mp.Manager(); ret = mgr.dict()
    mp.spawn(_tp_worker, args=(2, _free_port(), ret), nprocs=2, join=True)
    for rank in range(2):
        assert all(ret[rank]), ret[rank]


ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_starts_its_own_ranks():
    """`bench.py --gpus 2` without a launcher around it starts two ranks itself: here the launcher path alone
    (gloo, CPU tensors, the job reduction only).  The line reports the ranks that actually joined, the slowest
    rank's time and the sum of the units; the ranks hold disjoint global sequences."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_PORT")}
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--launcher-selftest"],
                       capture_output=True, text=True, timeout=300, cwd=ROOT, env=env)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, p.stdout                     # rank 0 alone prints
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["max_ms"] == 15.0 and d["units"] == 300.0 and d["value"] == 20000.0
    assert d["id_sum"] == sum(range(8))                  # sequences 0..3 on rank 0, 4..7 on rank 1


def test_bench_refuses_more_gpus_than_visible():
    """A plain `python bench.py --gpus N` on a machine with fewer than N devices must fail, not print n_gpus = N."""
    import torch
    n = (torch.cuda.device_count() if torch.cuda.is_available() else 0) + 1
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_PORT")}
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", str(max(n, 2)), "--steps", "1"],
                       capture_output=True, text=True, timeout=300, cwd=ROOT, env=env)
    assert p.returncode != 0 and "visible" in (p.stderr + p.stdout)
    assert not [l for l in p.stdout.splitlines() if l.startswith("{")]


def test_spawn_ranks_reports_a_failing_rank():
    code = "import os, sys, time; r = int(os.environ['RANK']); time.sleep(0.2 * r); sys.exit(3 if r == 1 else 0)"
    assert dist_util.spawn_ranks([sys.executable, "-c", code], 3) == 3
    assert dist_util.spawn_ranks([sys.executable, "-c", "import os; assert os.environ['WORLD_SIZE'] == '2'"], 2) == 0
