#!/usr/bin/env python
"""Benchmark of the Lethe hot path on B200: decode-step attention over the pruned KV cache (with the fused
relevance update) plus the prune round every `prune_interval` steps, on the Llama-8B-shaped workload.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" = one decode step of the whole model shape (all layers, one lethe_decode_attend call) and, when the
step index hits the prune interval, one prune round (estimate_sparsity -> alloc_budgets -> rasr_prune).  The
printed JSON line follows the driver's contract; `value` is KV token-heads attended per second with the cache
and the step inputs resident in HBM, `e2e` is the same through lethe_decode_attend_host (per-step q / k_new /
v_new in pinned host memory, out delivered to pinned host memory, a stream synchronise every step; with pinned
buffers the persistent kernel moves those bytes over the bus itself instead of through copies, see `transfer`).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2511_06029_b200 import dist_util, synth  # noqa: E402

METRIC = "kv_token_heads_attended_per_s"
UNIT = "token-heads/s"
BYTES_PER_TOKEN_HEAD = 520          # K row 256 B + V row 256 B + relevance read 4 B + write 4 B (D=128, bf16)
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes (read + write) per token-head of the default attend kernel, from the ncu capture summarised in
# profiles/attend_async_w8s2_llama8b.md (1.026 GB per launch of 1 969 552 token-heads; traffic grows in
# proportion to the token-heads of a launch, so it is scaled to the launch bench.py times).
NCU_TRAFFIC_BYTES_PER_TOKEN_HEAD = 521.0


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples of one GPU while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "50", "-i", str(gpu_index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1])); mx.append(float(parts[2]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def make_state(w, device, capacity, n0, seed):
    """Device-resident cache at n0 tokens per item, values drawn on the device (throughput-only tensors)."""
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    L, B, H, D = w.n_layers, w.batch, w.n_kv_heads, w.head_dim
    k = torch.empty((L, B, H, capacity, D), dtype=w.dtype, device=device)
    v = torch.empty((L, B, H, capacity, D), dtype=w.dtype, device=device)
    flags = synth.anchor_flags(w, torch.arange(capacity, device=device), torch.arange(B))   # [L][B][cap]
    for l in range(L):
        kk = torch.randn((B, H, capacity, D), generator=g, device=device, dtype=torch.float32)
        kk *= torch.where(flags[l], w.anchor_gain, 1.0).to(torch.float32)[:, None, :, None]
        k[l] = kk.to(w.dtype)
        v[l] = torch.randn((B, H, capacity, D), generator=g, device=device, dtype=torch.float32).to(w.dtype)
    rel = torch.zeros((L, B, H, capacity), dtype=torch.float32, device=device)
    pos = torch.arange(capacity, dtype=torch.int32, device=device).expand(L, B, H, capacity).contiguous()
    ln = torch.full((L, B, H), n0, dtype=torch.int32, device=device)
    return k, v, rel, pos, ln


class Runner:
    """The decode / prune loop around the C ABI (host logic of the harness: when to prune)."""

    def __init__(self, w, device, rank, capacity, variant, splits, pool=8, kv="bf16"):
        from paper_2511_06029_b200 import binding
        self.w, self.dev, self.binding = w, device, binding
        self.ctx = binding.Context(device.index)
        self.ctx.set_tuning(variant, splits)
        k, v, rel, pos, ln = make_state(w, device, capacity, w.mean_budget, 1234 + 77 * rank)
        if kv != "bf16":   # quantised cache: bytes, one scale per layer (anchor keys reach about 3 x 4 sigma)
            f8, fmax = (torch.float8_e4m3fn, 448.0) if kv == "fp8" else (torch.float8_e5m2, 57344.0)
            ks, vs = [0.125] * w.n_layers, [0.0625] * w.n_layers
            k = (k.float() / ks[0]).clamp(-fmax, fmax).to(f8)
            v = (v.float() / vs[0]).clamp(-fmax, fmax).to(f8)
            self.cache = binding.Cache(w.n_q_heads, k, v, rel, pos, ln, k_scale=ks, v_scale=vs)
        else:
            self.cache = binding.Cache(w.n_q_heads, k, v, rel, pos, ln)
        self.scale = synth.layer_scales(w).tolist()
        self.scale_c = self.ctx._scale(self.scale)
        L, B = w.n_layers, w.batch
        g = torch.Generator(device=device); g.manual_seed(4321 + rank)
        self.pool = []
        for i in range(pool):
            q = torch.randn((L, B, w.n_q_heads, w.head_dim), generator=g, device=device).to(w.dtype)
            kn = torch.randn((L, B, w.n_kv_heads, w.head_dim), generator=g, device=device).to(w.dtype)
            vn = torch.randn((L, B, w.n_kv_heads, w.head_dim), generator=g, device=device).to(w.dtype)
            self.pool.append((q, kn, vn))
        # pinned host copies of the same inputs: the end-to-end loop replays exactly the device loop's sequence
        self.host_pool = [tuple(t.cpu().pin_memory() for t in p) for p in self.pool]
        self.out = torch.empty((L, B, w.n_q_heads, w.head_dim), dtype=w.dtype, device=device)
        self.out_host = torch.empty((L, B, w.n_q_heads, w.head_dim), dtype=w.dtype).pin_memory()
        self.token_pos = torch.zeros((B,), dtype=torch.int32, device=device)
        self.token_pos_host = torch.zeros((B,), dtype=torch.int32).pin_memory()
        self.S = torch.zeros((L, B), dtype=torch.float32, device=device)
        self.budgets = torch.zeros((L, B), dtype=torch.int32, device=device)
        self.T = torch.full((B,), w.total_budget, dtype=torch.int64, device=device)
        self.step_no = 0
        self.launches = 0

    def decode(self, host=False):
        w = self.w
        i = self.step_no
        if host:
            q, kn, vn = self.host_pool[i % len(self.host_pool)]
            self.ctx.decode_attend_host(self.cache, 0, w.n_layers, q, kn, vn, self.token_pos_host, self.scale, w.gamma,
                                        self.out_host, None, scale_c=self.scale_c)
        else:
            q, kn, vn = self.pool[i % len(self.pool)]
            self.ctx.decode_attend(self.cache, 0, w.n_layers, q, kn, vn, self.token_pos, self.scale, w.gamma, self.out,
                                   None, scale_c=self.scale_c)
        self.launches += 1
        self.step_no += 1

    def prune_due(self):
        return self.step_no % self.w.prune_interval == 0

    def prune(self):
        w = self.w
        self.ctx.estimate_sparsity(self.cache, self.S)
        self.ctx.alloc_budgets(self.S, self.T, w.k_min, self.budgets)
        self.ctx.rasr_prune(self.cache, self.budgets, w.recent, w.sink)
        self.launches += 3

    def check(self):
        st, item = self.ctx.poll_status()
        if st != 0:
            raise RuntimeError(f"device-side status {st} at item {item}")


def timed_loop(r: Runner, steps: int, host: bool):
    """Run `steps` steps; returns (total_ms, attend_ms list, prune_ms list, token_heads list)."""
    dev = r.dev
    stream = torch.cuda.current_stream(dev)
    ev = [] if host else [torch.cuda.Event(enable_timing=True) for _ in range(2 * steps)]   # per-launch times: device loop only
    prune_ev = []
    len_snap = [(0, r.cache.len.clone())]
    t_begin = torch.cuda.Event(enable_timing=True); t_end = torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(dev)
    t_begin.record(stream)
    for s in range(steps):
        if host:
            r.decode(host=True)
            stream.synchronize()               # the caller reads out before producing the next token
        else:
            ev[2 * s].record(stream)
            r.decode(host=False)
            ev[2 * s + 1].record(stream)
        if r.prune_due():
            a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            a.record(stream)
            r.prune()
            b.record(stream)
            prune_ev.append((a, b))
            snap = torch.empty_like(r.cache.len)
            snap.copy_(r.cache.len, non_blocking=True)
            len_snap.append((s + 1, snap))
    t_end.record(stream)
    torch.cuda.synchronize(dev)
    total_ms = t_begin.elapsed_time(t_end)
    attend_ms = [] if host else [ev[2 * s].elapsed_time(ev[2 * s + 1]) for s in range(steps)]
    prune_ms = [a.elapsed_time(b) for a, b in prune_ev]
    # token-heads attended at step s = sum of len after that step's append
    items = r.cache.len.numel()
    th = []
    snaps = [(s0, int(t.sum().item())) for s0, t in len_snap]
    for s in range(steps):
        base_step, base_sum = max((x for x in snaps if x[0] <= s), key=lambda x: x[0])
        th.append(base_sum + items * (s - base_step + 1))
    return total_ms, attend_ms, prune_ms, th


def per_layer_mode(r: Runner, steps: int):
    """The same decode step issued the way a real model must (layer l+1's query does not exist before layer l
    is done): one lethe_decode_attend launch per layer, the 32 launches replayed from a CUDA graph.  Returns
    (ms per step, token-heads per step)."""
    w, dev = r.w, r.dev
    q, kn, vn = r.pool[0]

    def one_step():
        for l in range(w.n_layers):
            r.ctx.decode_attend(r.cache, l, l + 1, q[l:l + 1], kn[l:l + 1], vn[l:l + 1], r.token_pos, r.scale, w.gamma,
                                r.out[l:l + 1], None, scale_c=r.scale_c)

    side = torch.cuda.Stream(dev)
    side.wait_stream(torch.cuda.current_stream(dev))
    with torch.cuda.stream(side):
        one_step()                                   # first use of this kernel outside capture
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            one_step()
    torch.cuda.current_stream(dev).wait_stream(side)
    torch.cuda.synchronize(dev)
    th0 = int(r.cache.len.sum().item())
    items = r.cache.len.numel()
    a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
    for _ in range(3):
        graph.replay()
    a.record()
    for _ in range(steps):
        graph.replay()
    b.record()
    torch.cuda.synchronize(dev)
    ms = a.elapsed_time(b) / steps
    th = th0 + items * (3 + (steps + 1) / 2.0)       # mean length over the timed replays
    return ms, th


def cpu_baseline(w, r: Runner | None, seconds=12.0, layers=8, seqs=4):
    """The oracle, as it stands, on a bounded sample of the workload on the host cores."""
    import oracle
    threads = oracle.max_threads()
    oracle.set_threads(threads)
    ws = synth.shrink(w, n_layers=layers, batch=seqs)
    max_steps = 600
    cap = w.mean_budget + max_steps + 8
    st = synth.initial_kv(ws, w.mean_budget, cap)
    oc = oracle.OracleCache(ws.n_layers, seqs, ws.n_q_heads, ws.n_kv_heads, ws.head_dim, cap, st["k"], st["v"],
                            st["rel"], st["pos"], st["len"])
    scale = synth.layer_scales(w)[:layers].contiguous()
    th = 0
    t0 = time.perf_counter()
    steps = 0
    while True:
        x = synth.step_inputs(ws, steps)
        t1 = time.perf_counter()
        s, *_ = oracle.decode_attend(oc, 0, layers, x["q"], x["k_new"], x["v_new"], x["token_pos"], scale, w.gamma)
        dt = time.perf_counter() - t1
        assert s == oracle.OK
        th += int(oc.len.sum())
        steps += 1
        if steps == 1:
            first = dt
        if time.perf_counter() - t0 > seconds or steps >= max_steps - 90:
            break
    attend_s = time.perf_counter() - t0
    # one prune round on the sample, amortised like the GPU loop
    t1 = time.perf_counter()
    _, S = oracle.estimate_sparsity(oc)
    _, bud = oracle.alloc_budgets(S, torch.full((seqs,), layers * w.mean_budget, dtype=torch.int64), w.k_min)
    oracle.rasr_prune(oc, bud, w.recent, w.sink)
    prune_s = time.perf_counter() - t1
    per_step = attend_s / steps + prune_s / w.prune_interval
    overlap = None
    if r is not None:
        overlap = retained_set_overlap(w, ws, r.dev, oc, cap, steps, layers, seqs, scale)
    # the same oracle on one core, on a few more steps of the same sample (decode only; the prune share is ~1 %)
    oracle.set_threads(1)
    t1 = time.perf_counter()
    th1 = 0
    n1 = 0
    while time.perf_counter() - t1 < 3.0 and steps + n1 < max_steps - 1:
        x = synth.step_inputs(ws, steps + n1)
        s, *_ = oracle.decode_attend(oc, 0, layers, x["q"], x["k_new"], x["v_new"], x["token_pos"], scale, w.gamma)
        assert s == oracle.OK
        th1 += int(oc.len.sum())
        n1 += 1
    one_core = th1 / (time.perf_counter() - t1) if n1 else None
    oracle.set_threads(threads)
    return {"value": th / steps / per_step, "unit": UNIT, "cores": threads, "kind": "oracle", "value_1_core": one_core,
            "sample": f"{layers} layers x {seqs} sequences x {w.n_kv_heads} KV heads at ~{w.mean_budget} tokens, "
                      f"{steps} decode steps in {attend_s:.1f} s plus one prune round ({prune_s * 1e3:.0f} ms) "
                      f"amortised over {w.prune_interval} steps",
            "ms_per_sample_step": per_step * 1e3, "token_heads_per_sample_step": th / steps,
            "retained_set_overlap": overlap}


def retained_set_overlap(w, ws, dev, oc, cap, steps, layers, seqs, scale):
    """End-to-end agreement of what is kept: the GPU path replays the sample the oracle was just timed on (same
    initial cache, same per-step inputs, same number of steps, then one prune round), free-running on its own
    scores, and the retained positions of every item are compared with the oracle's."""
    from paper_2511_06029_b200 import binding
    st = synth.initial_kv(ws, w.mean_budget, cap)
    gc = binding.Cache(ws.n_q_heads, *(st[k].to(dev) for k in ("k", "v", "rel", "pos", "len")))
    ctx = binding.Context(dev.index)
    try:
        sc = scale.tolist()
        out = torch.empty((layers, seqs, ws.n_q_heads, ws.head_dim), dtype=ws.dtype, device=dev)
        for i in range(steps):
            x = synth.step_inputs(ws, i)
            ctx.decode_attend(gc, 0, layers, x["q"].to(dev), x["k_new"].to(dev), x["v_new"].to(dev),
                              x["token_pos"].to(dev), sc, w.gamma, out)
        S = torch.zeros((layers, seqs), dtype=torch.float32, device=dev)
        bud = torch.zeros((layers, seqs), dtype=torch.int32, device=dev)
        T = torch.full((seqs,), layers * w.mean_budget, dtype=torch.int64, device=dev)
        ctx.estimate_sparsity(gc, S)
        ctx.alloc_budgets(S, T, w.k_min, bud)
        ctx.rasr_prune(gc, bud, w.recent, w.sink)
        status, _ = ctx.poll_status()
        glen, gpos = gc.len.cpu(), gc.pos.cpu()
    finally:
        ctx.close()
    jac, same = [], 0
    for l in range(layers):
        for b in range(seqs):
            for h in range(ws.n_kv_heads):
                a = set(gpos[l, b, h, :int(glen[l, b, h])].tolist())
                o = set(oc.pos[l, b, h, :int(oc.len[l, b, h])].tolist())
                jac.append(len(a & o) / max(1, len(a | o)))
                same += a == o
    return {"items": len(jac), "decode_steps": steps, "device_status": status,
            "jaccard_mean": sum(jac) / len(jac), "jaccard_min": min(jac), "identical_sets": same / len(jac),
            "equal_lengths": float((glen == oc.len).float().mean()),
            "note": "GPU free-running on its own fp32 scores vs the oracle (fp64), retained positions per (layer, sequence, KV head) "
                    "after the sample's decode steps and one prune round"}


def run_reference(args, w):
    """--impl reference: the oracle on the host cores, same metric / config keys."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    base = cpu_baseline(w, None, seconds=max(5.0, min(60.0, 0.5 * (args.steps + args.warmup))))
    line = {"impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": base["ms_per_sample_step"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w, args, extra={"note": "oracle timed on a bounded sample per step"}),
            "cpu_baseline": base,
            "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def workload_config(w, args, extra=None):
    c = {"workload": f"{w.name}: L{w.n_layers} B{w.batch} Hq{w.n_q_heads}/Hkv{w.n_kv_heads} D{w.head_dim} bf16, "
                     f"mean budget {w.mean_budget}/layer, recent {w.recent}, sink {w.sink}, prune every "
                     f"{w.prune_interval} steps, gamma {w.gamma}",
         "global_batch": w.batch * args.gpus, "l2": "inputs larger than L2 (>=1.1 GB of K/V streamed per step)",
         "parallelism": f"dp{args.gpus} (sequences sharded, no data-path collective)"}
    if extra:
        c.update(extra)
    return c


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1024)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama8b")
    ap.add_argument("--variant", type=int, default=0)
    ap.add_argument("--splits", type=int, default=0)
    ap.add_argument("--capacity", type=int, default=0)
    ap.add_argument("--prep-rounds", type=int, default=6,
                    help="untimed prune intervals run before warm-up so that lengths reach their budgets")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-per-layer", action="store_true")
    ap.add_argument("--kv", choices=["bf16", "fp8", "fp8e5m2"], default="bf16",
                    help="storage of K and V: bf16 (the headline configuration), or e4m3 / e5m2 bytes with per-layer scales")
    ap.add_argument("--with-prefill", action="store_true",
                    help="also time lethe_prefill_seed on a prompt of the workload's length (informational)")
    ap.add_argument("--pl-variant", type=int, default=0, help="kernel variant of the per-layer launch mode")
    ap.add_argument("--pl-splits", type=int, default=0)
    args = ap.parse_args()
    w = synth.WORKLOADS[args.workload]

    if args.impl == "reference":
        run_reference(args, w)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    dist = None
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    from paper_2511_06029_b200 import build
    if rank == 0 or world == 1:
        build.build()
    if dist is not None:
        dist.barrier()

    # algorithmic bytes per token-head: K row + V row + relevance read and write (rows are D bytes when quantised)
    bytes_per_th = BYTES_PER_TOKEN_HEAD if args.kv == "bf16" else 2 * w.head_dim + 8

    def prepare(capacity):
        """Runner brought to steady state (untimed): a few full prune intervals so that relevance, sparsity-driven
        budgets and lengths are those of a long trajectory (dense layers need several rounds to grow to their
        budget).  Returns the runner and the largest layer budget."""
        r = Runner(w, dev, rank, capacity, args.variant, args.splits, kv=args.kv)
        for _ in range(max(1, args.prep_rounds)):
            for _ in range(w.prune_interval):
                r.decode()
            r.prune()
        r.check()
        return r, int(r.budgets.max().item())

    # Capacity = largest layer budget + prune interval (+ slack), as a serving system would size it.  The budgets
    # follow from the measured sparsity, so a pilot run at a generous capacity finds them first.
    if args.capacity:
        capacity = args.capacity
        r, max_budget = prepare(capacity)
    else:
        pilot, max_budget = prepare(3 * w.mean_budget)
        pilot.ctx.close()
        del pilot
        torch.cuda.empty_cache()
        capacity = -(-(max_budget + w.prune_interval + 32) // 64) * 64
        r, max_budget = prepare(capacity)
    if max_budget + w.prune_interval > capacity:
        raise SystemExit(f"capacity {capacity} too small for budget {max_budget} + interval {w.prune_interval}")
    for _ in range(max(args.warmup, 3)):
        r.decode()
        if r.prune_due():
            r.prune()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    sampler = ClockSampler(local) if rank == 0 else None
    barrier()
    r.launches = 0
    total_ms, attend_ms, prune_ms, th = timed_loop(r, args.steps, host=False)
    launches = r.launches
    barrier()
    r.check()
    e2e = None
    if not args.no_e2e:
        barrier()
        e_total_ms, _, _, e_th = timed_loop(r, args.steps, host=True)
        barrier()
        r.check()
    clocks = sampler.stop() if sampler else None
    per_layer = None
    if not args.no_per_layer and world == 1:
        pl_steps = min(32, max(4, w.prune_interval - (r.step_no % w.prune_interval) - 8))
        r.ctx.set_tuning(args.pl_variant, args.pl_splits)
        ms_pl, th_pl = per_layer_mode(r, pl_steps)
        r.ctx.set_tuning(args.variant, args.splits)
        r.check()
        per_layer = {"ms_per_step": ms_pl, "token_heads_per_step": th_pl, "value": th_pl / (ms_pl * 1e-3),
                     "algorithmic_GBs": th_pl * bytes_per_th / (ms_pl * 1e-3) / 1e9,
                     "mode": f"{w.n_layers} launches per step (one per layer), replayed from a CUDA graph, "
                             f"{pl_steps} steps; not part of `value`"}

    # Retention by the collapsed score of Eq. 2 (one set per sequence), timed once on the live state with the
    # budgets a RASR round would get now: the row traffic of such a round.  Only the heads' lengths are aligned here (the
    # earlier rounds pruned head by head), so this is a timing of the call, not a meaningful retention.
    collapsed = None
    if not args.no_per_layer and world == 1:
        from paper_2511_06029_b200 import binding as _b
        r.ctx.estimate_sparsity(r.cache, r.S)
        r.ctx.alloc_budgets(r.S, r.T, w.k_min, r.budgets)
        before = int(r.cache.len.sum().item())
        a_ev = torch.cuda.Event(enable_timing=True); b_ev = torch.cuda.Event(enable_timing=True)
        a_ev.record()
        r.ctx.collapsed_prune(r.cache, r.budgets, w.recent, w.sink, _b.COLLAPSE_HEADS)
        b_ev.record()
        torch.cuda.synchronize(dev)
        r.check()
        collapsed = {"scope": "heads (one set per layer and sequence)", "ms": a_ev.elapsed_time(b_ev),
                     "token_heads_before": before, "token_heads_after": int(r.cache.len.sum().item())}

    # Algorithm 1 (threshold-triggered, budget-free retention) timed once on the live state, after everything
    # that enters `value`: first with the paper's default sparse_ratio (tau = 400), then with a small tau that
    # does find breakpoints and therefore also compacts.
    segment = None
    if not args.no_per_layer and world == 1:
        le = torch.zeros_like(r.cache.len)
        segment = {}
        for tau in (400.0, 4.0):
            le.zero_()
            before = int(r.cache.len.sum().item())
            a_ev = torch.cuda.Event(enable_timing=True); b_ev = torch.cuda.Event(enable_timing=True)
            a_ev.record()
            r.ctx.segment_prune(r.cache, 8, tau, w.recent, w.sink, le)
            b_ev.record()
            torch.cuda.synchronize(dev)
            segment[f"tau_{int(tau)}"] = {"ms": a_ev.elapsed_time(b_ev), "token_heads_before": before,
                                          "token_heads_after": int(r.cache.len.sum().item())}
        r.check()
    prefill = None
    if args.with_prefill and world == 1:
        from paper_2511_06029_b200 import binding
        P = w.prompt_len
        gq = torch.Generator(device=dev); gq.manual_seed(99)
        kp = torch.randn((w.n_layers, w.batch, w.n_kv_heads, P, w.head_dim), generator=gq, device=dev).to(w.dtype)
        pc = binding.Cache(w.n_q_heads, kp, torch.zeros_like(kp),
                           torch.zeros((w.n_layers, w.batch, w.n_kv_heads, P), device=dev),
                           torch.zeros((w.n_layers, w.batch, w.n_kv_heads, P), dtype=torch.int32, device=dev),
                           torch.full((w.n_layers, w.batch, w.n_kv_heads), P, dtype=torch.int32, device=dev))
        qp = torch.randn((w.n_layers, w.batch, P, w.n_q_heads, w.head_dim), generator=gq, device=dev).to(w.dtype)
        flops = 2.0 * pc.len.numel() * w.group * (P * (P + 1) / 2) * w.head_dim * 2   # two passes over the causal half
        exps = 2.0 * pc.len.numel() * w.group * (P * (P + 1) / 2)                      # one exponential per logit and pass
        peaks = {}
        try:
            peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        except Exception:
            pass
        xu_peak = 148 * 16 * peaks.get("sm_max_mhz", 1965.0) * 1e6                      # ex2 per second: 16 per SM per clock
        engines = {}
        for name_e, code in (("tcgen05", 40), ("mma_sync", 41)):
            r.ctx.set_tuning(code, 0)
            for _ in range(2):
                r.ctx.prefill_seed(pc, qp, r.scale, w.gamma)
            a_ev = torch.cuda.Event(enable_timing=True); b_ev = torch.cuda.Event(enable_timing=True)
            a_ev.record()
            for _ in range(5):
                r.ctx.prefill_seed(pc, qp, r.scale, w.gamma)
            b_ev.record()
            torch.cuda.synchronize(dev)
            r.check()
            ms_p = a_ev.elapsed_time(b_ev) / 5
            tf = flops / (ms_p * 1e-3) / 1e12
            engines[name_e] = {"ms": ms_p, "useful_TFLOPs": tf,
                               "frac_of_measured_bf16_burst": (tf / peaks["bf16_tflops"]) if "bf16_tflops" in peaks else None,
                               "frac_of_ex2_peak": exps / (ms_p * 1e-3) / xu_peak}
        r.ctx.set_tuning(40, 0)
        prefill = {"prompt_len": P, "engines": engines, "bound": "alu (ex2: one exponential per logit and pass)",
                   "ex2_peak_per_s": xu_peak,
                   "note": "two passes (statistics, column sums), 2 launches per call; tcgen05 = default engine "
                           "(accumulators in tensor memory, TMA operand tiles), mma_sync = the legacy tensor path"}
        del pc, kp, qp
    e_ms = e_total_ms if not args.no_e2e else 0.0
    e_u = float(sum(e_th)) if not args.no_e2e else 0.0
    (t_ms, e_total_ms), (units, e_units) = dist_util.reduce_job(dist, dev, [total_ms, e_ms], [float(sum(th)), e_u])

    if rank == 0:
        peak, which = measured_peak()
        th_per_launch = sum(th) / len(th)
        avg_attend_ms = sum(attend_ms) / len(attend_ms)
        achieved = th_per_launch * bytes_per_th / (avg_attend_ms * 1e-3) / 1e9
        wq = w
        h2d = (wq.n_layers * wq.batch * (wq.n_q_heads + 2 * wq.n_kv_heads) * wq.head_dim * 2 + wq.batch * 4)
        d2h = wq.n_layers * wq.batch * wq.n_q_heads * wq.head_dim * 2
        line = {
            "metric": METRIC, "value": dist_util.job_value(units, t_ms), "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": t_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if args.kv == "bf16" else
                     f"fp8 K/V ({'e4m3' if args.kv == 'fp8' else 'e5m2'} bytes, per-layer scales), bf16 activations, f16 mma, fp32 accumulation",
            "data": "synthetic",
            "config": workload_config(w, args, extra={
                "capacity": capacity, "variant": args.variant, "splits": args.splits,
                "launch_mode": "all layers in one lethe_decode_attend call per step",
                "token_heads_per_step": th_per_launch,
                "prune_rounds_timed": len(prune_ms),
                "prune_round_ms": (sum(prune_ms) / len(prune_ms)) if prune_ms else None,
                "attend_ms_per_step": avg_attend_ms,
                "attend_ms_median": statistics.median(attend_ms),
                "per_layer_launch": per_layer,
                "segment_prune_8_segments": segment,
                "collapsed_prune": collapsed,
                "prefill_seed": prefill}),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "peak_source": f"of {which}", "frac_of_8TBs_nominal": achieved / 8000.0,
                         "kernel": "attend (dominant kernel; one launch per step)",
                         "traffic": (NCU_TRAFFIC_BYTES_PER_TOKEN_HEAD * th_per_launch
                                     if (NCU_TRAFFIC_BYTES_PER_TOKEN_HEAD and args.kv == "bf16") else None)},
            "gpu_launches": launches, "clocks": clocks,
        }
        if not args.no_e2e:
            line["e2e"] = {"value": dist_util.job_value(e_units, e_total_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
                           "d2h_bytes_per_step": d2h, "ms_per_step": e_total_ms / args.steps,
                           "transfer": "pinned host buffers; the attend kernel reads the step's inputs from them and "
                                       "writes out into them over the bus, inside the timed launch (pageable buffers "
                                       "would take staged copies)"}
        if not args.no_cpu_baseline and world == 1:   # the oracle is timed beside the single-GPU run only
            line["cpu_baseline"] = cpu_baseline(w, r)
            line["retained_set_overlap"] = line["cpu_baseline"].pop("retained_set_overlap", None)
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
