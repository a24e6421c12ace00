#!/usr/bin/env python
"""Benchmark of the Lethe hot path on B200: decode-step attention over the pruned KV cache (with the fused
relevance update) plus the prune round every `prune_interval` steps.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--workload llama8b|qwen7b|longreason|ragged] [--sweep]

One "step" = one decode step of the whole model shape (all resident layers, one lethe_decode_attend call) and,
when the step index hits the prune interval, one prune round (estimate_sparsity -> alloc_budgets -> rasr_prune).
The printed JSON line follows the driver's contract:
  value / ms_per_step  the K timed steps as they ran, cache and step inputs resident in HBM;
  e2e                  the same through lethe_decode_attend_host (per-step q / k_new / v_new in pinned host
                       memory, out delivered to pinned host memory, a stream synchronise every step);
  config.prune_round   the prune round, timed on every run whatever K is: at least three full rounds after the
                       timed loop (a prune interval of untimed decode steps before each), the three calls timed
                       one by one, with its amortised cost per decode step and the roofline of the decode step
                       plus that amortised share.
With --gpus N > 1 and no launcher in the environment, bench.py starts the N ranks itself (one process per GPU);
under torchrun it uses the ranks it is given.  Sequences are sharded across ranks; no collective touches the data
path.
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
NOMINAL_HBM_GBS = 8000.0
# DRAM bytes (read + write) per token-head of the attend kernel each workload runs by default, from the ncu
# captures summarised under profiles/ (traffic grows in proportion to the token-heads of a launch, so the
# per-token-head figure of the capture is scaled to the launch bench.py times).  None = no capture on record.
NCU_TRAFFIC = {
    "llama8b": (519.8, "profiles/attend_async_w8s2_llama8b_bench.md"),
    "qwen7b": (521.5, "profiles/attend_stream_w8s2_qwen7b.md"),
    "longreason": (519.1, "profiles/attend_async_spill_w8s2_longreason.md"),
    "ragged": (520.5, "profiles/attend_stream_paged_w8s2_ragged.md"),
    "llama8b:fp8": (267.5, "profiles/attend_kv8_tc_llama8b.md"),
}
RAGGED_RESIDENT_LAYERS = 7           # of 28: the full ragged state is 124 GB of K/V; one layer group is resident at a time
SWEEP_RATIOS = (0.05, 0.1, 0.25, 0.5)
SWEEP_INTERVALS = (64, 256, 1024)


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


# ----------------------------------------------------------------------------------------- synthetic state

def make_state(w, device, capacity, n0, seed, batch_ids):
    """Device-resident contiguous cache at n0 tokens per item for the global sequences `batch_ids`, values drawn
    on the device (throughput-only tensors)."""
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    L, B, H, D = w.n_layers, int(batch_ids.numel()), w.n_kv_heads, w.head_dim
    k = torch.empty((L, B, H, capacity, D), dtype=w.dtype, device=device)
    v = torch.empty((L, B, H, capacity, D), dtype=w.dtype, device=device)
    flags = synth.anchor_flags(w, torch.arange(capacity, device=device), batch_ids)   # [L][B][cap]
    for l in range(L):
        kk = torch.randn((B, H, capacity, D), generator=g, device=device, dtype=torch.float32)
        kk *= torch.where(flags[l], w.anchor_gain, 1.0).to(torch.float32)[:, None, :, None]
        k[l] = kk.to(w.dtype)
        v[l] = torch.randn((B, H, capacity, D), generator=g, device=device, dtype=torch.float32).to(w.dtype)
    rel = torch.zeros((L, B, H, capacity), dtype=torch.float32, device=device)
    pos = torch.arange(capacity, dtype=torch.int32, device=device).expand(L, B, H, capacity).contiguous()
    ln = torch.full((L, B, H), n0, dtype=torch.int32, device=device)
    return k, v, rel, pos, ln, None


def make_state_ragged(w, device, lens_seq, cap_pages, seed):
    """Device-resident paged cache (16-token pages, one shuffled page table per item) whose sequence b holds
    lens_seq[b] tokens in every layer and head.  The pools hold only the pages a sequence can reach
    (ceil((cap tokens it may grow to) / 16) per item); table entries beyond that point at a spare page."""
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    L, B, H, D, pt = w.n_layers, int(lens_seq.numel()), w.n_kv_heads, w.head_dim, w.page_tokens
    reach = torch.clamp((lens_seq + max(SWEEP_INTERVALS) + 2 * pt + pt - 1) // pt, max=cap_pages)   # pages per item of sequence b
    per_item = reach[None, :, None].expand(L, B, H).reshape(-1)
    n_pages = int(per_item.sum().item()) + 1                       # + the spare page (id n_pages - 1)
    k = torch.empty((n_pages, pt, D), dtype=w.dtype, device=device)
    v = torch.empty((n_pages, pt, D), dtype=w.dtype, device=device)
    chunk = 1 << 15
    for i in range(0, n_pages, chunk):
        m = min(chunk, n_pages - i)
        k[i:i + m] = torch.randn((m, pt, D), generator=g, device=device).to(w.dtype)
        v[i:i + m] = torch.randn((m, pt, D), generator=g, device=device).to(w.dtype)
    perm = torch.randperm(n_pages - 1, generator=g, device=device).to(torch.int32)   # fragmented on purpose
    table = torch.full((L * B * H, cap_pages), n_pages - 1, dtype=torch.int32, device=device)
    col = torch.arange(cap_pages, device=device)[None, :]
    mask = col < per_item.to(device)[:, None]
    table[mask] = perm[: int(mask.sum().item())]
    table = table.reshape(L, B, H, cap_pages).contiguous()
    cap_tokens = cap_pages * pt
    rel = torch.zeros((L, B, H, cap_tokens), dtype=torch.float32, device=device)
    pos = torch.arange(cap_tokens, dtype=torch.int32, device=device).expand(L, B, H, cap_tokens).contiguous()
    ln = lens_seq.to(torch.int32).to(device)[None, :, None].expand(L, B, H).contiguous()
    return k, v, rel, pos, ln, table


class Runner:
    """The decode / prune loop around the C ABI (host logic of the harness: when to prune)."""

    def __init__(self, w, device, rank, capacity, variant, splits, pool=8, kv="bf16", lens_seq=None, total_budget=None):
        from paper_2511_06029_b200 import binding
        self.w, self.dev, self.binding = w, device, binding
        self.ctx = binding.Context(device.index)
        self.ctx.set_tuning(variant, splits)
        self.batch_ids = dist_util.rank_batch_ids(rank, w.batch)    # the global sequences this rank holds
        seed = 1234 + 77 * int(self.batch_ids[0])
        if w.page_tokens:
            k, v, rel, pos, ln, table = make_state_ragged(w, device, lens_seq, capacity, seed)
        else:
            k, v, rel, pos, ln, table = make_state(w, device, capacity, w.mean_budget, seed, self.batch_ids)
        if kv != "bf16":   # quantised cache: bytes, one scale per layer (anchor keys reach about 3 x 4 sigma)
            f8, fmax = (torch.float8_e4m3fn, 448.0) if kv == "fp8" else (torch.float8_e5m2, 57344.0)
            ks, vs = [0.125] * w.n_layers, [0.0625] * w.n_layers
            k = (k.float() / ks[0]).clamp(-fmax, fmax).to(f8)
            v = (v.float() / vs[0]).clamp(-fmax, fmax).to(f8)
            self.cache = binding.Cache(w.n_q_heads, k, v, rel, pos, ln, table, k_scale=ks, v_scale=vs)
        else:
            self.cache = binding.Cache(w.n_q_heads, k, v, rel, pos, ln, table)
        self.scale = synth.layer_scales(w).tolist()
        self.scale_c = self.ctx._scale(self.scale)
        L, B = w.n_layers, w.batch
        g = torch.Generator(device=device); g.manual_seed(4321 + int(self.batch_ids[0]))
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
        if total_budget is None:
            total_budget = torch.full((B,), w.total_budget, dtype=torch.int64)
        self.T = total_budget.to(torch.int64).to(device)
        self.step_no = 0
        self.launches = 0
        self.epoch = 0                                   # anchor draw in force (drifting workloads)

    def drift_if_due(self):
        """Untimed harness work of a drifting workload: when the step counter has crossed a drift period, the anchor
        set is re-drawn and the K rows whose flag changed are rescaled (rows are found through pos)."""
        e = synth.drift_epoch(self.w, self.step_no)
        if e != self.epoch and self.cache.page_table is None and self.cache.k.dtype == self.w.dtype:
            synth.apply_drift(self.w, self.cache.k, self.cache.pos, self.batch_ids, self.epoch, e)
        self.epoch = e

    def decode(self, host=False, append=True):
        w = self.w
        i = self.step_no
        if host:
            q, kn, vn = self.host_pool[i % len(self.host_pool)]
            self.ctx.decode_attend_host(self.cache, 0, w.n_layers, q, kn, vn, self.token_pos_host, self.scale, w.gamma,
                                        self.out_host, None, scale_c=self.scale_c)
        else:
            q, kn, vn = self.pool[i % len(self.pool)]
            if not append:
                kn = vn = None
            self.ctx.decode_attend(self.cache, 0, w.n_layers, q, kn, vn, self.token_pos if append else None, self.scale,
                                   w.gamma, self.out, None, scale_c=self.scale_c)
        self.launches += 1
        if append:
            self.step_no += 1

    def prune_due(self):
        return self.step_no % self.w.prune_interval == 0

    def prune(self, events=None, keep_idx=None):
        """One prune round; with `events` (4 CUDA events) the three calls are bracketed one by one."""
        w = self.w
        stream = torch.cuda.current_stream(self.dev)
        if events: events[0].record(stream)
        self.ctx.estimate_sparsity(self.cache, self.S)
        if events: events[1].record(stream)
        self.ctx.alloc_budgets(self.S, self.T, w.k_min, self.budgets)
        if events: events[2].record(stream)
        self.ctx.rasr_prune(self.cache, self.budgets, w.recent, w.sink, keep_idx)
        if events: events[3].record(stream)
        self.launches += 3

    def check(self):
        st, item = self.ctx.poll_status()
        if st != 0:
            raise RuntimeError(f"device-side status {st} at item {item}")

    def close(self):
        self.ctx.close()


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


def time_prune_rounds(r: Runner, rounds: int, bytes_per_th: int, attend_ms: float, th_per_step: float, peak: float):
    """The prune round of Sec. 4.1-4.3 on its own clock: `rounds` full rounds, each after decoding up to the next
    multiple of the prune interval (untimed), the three calls bracketed by CUDA events one by one.  One extra round
    before them (untimed, with keep_idx) counts the rows a round moves, from which the round's algorithmic bytes
    follow: relevance read once by the sparsity estimate and once by the selection (4 B each per token-head), and
    every survivor whose slot changes read and written once (K row + V row + relevance + position, twice)."""
    w, dev = r.w, r.dev
    row_bytes = bytes_per_th                              # a moved survivor: K row + V row + relevance 4 B + position 4 B

    def fill_interval():
        r.drift_if_due()
        while True:
            r.decode()
            if r.prune_due():
                break

    fill_interval()
    n_before = int(r.cache.len.sum().item())
    max_k = int(r.cache.len.max().item())
    keep = torch.empty((*r.cache.len.shape, max_k), dtype=torch.int32, device=dev)
    r.prune(keep_idx=keep)
    torch.cuda.synchronize(dev)
    idx = torch.arange(max_k, device=dev, dtype=torch.int32)
    moved = int(((keep >= 0) & (keep != idx)).sum().item())
    n_after = int(r.cache.len.sum().item())
    del keep
    parts = []
    for _ in range(rounds):
        fill_interval()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        r.prune(events=ev)
        torch.cuda.synchronize(dev)
        parts.append([ev[i].elapsed_time(ev[i + 1]) for i in range(3)])
    r.check()
    sp, bu, ra = (sum(p[i] for p in parts) / len(parts) for i in range(3))
    round_ms = sp + bu + ra
    round_bytes = 8 * n_before + 2 * row_bytes * moved
    amort_ms = round_ms / w.prune_interval
    step_ms = attend_ms + amort_ms
    step_gbs = th_per_step * bytes_per_th / (step_ms * 1e-3) / 1e9
    return {
        "rounds_timed": rounds, "prune_round_us": round_ms * 1e3,
        "estimate_sparsity_us": sp * 1e3, "alloc_budgets_us": bu * 1e3, "rasr_prune_us": ra * 1e3,
        "prune_amortised_us_per_step": amort_ms * 1e3, "prune_interval": w.prune_interval,
        "token_heads_before": n_before, "token_heads_after": n_after, "rows_moved": moved,
        "algorithmic_bytes": round_bytes,
        "roofline": {"bound": "hbm", "achieved": round_bytes / (round_ms * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                     "frac": round_bytes / (round_ms * 1e-3) / 1e9 / peak,
                     "bytes": "8 B per token-head before the round (relevance read by the sparsity estimate and by the "
                              "selection) + 2 x (K row + V row + 8 B) per survivor whose slot changes"},
        "decode_attend_plus_amortised_prune": {
            "ms_per_step": step_ms, "value": th_per_step / (step_ms * 1e-3), "unit": UNIT,
            "achieved": step_gbs, "frac": step_gbs / peak, "frac_of_8TBs_nominal": step_gbs / NOMINAL_HBM_GBS,
            "note": "attend launch (CUDA events, mean of the timed steps) + prune round / prune interval; bytes counted: "
                    "the attend's algorithmic bytes only"}}


def per_layer_mode(r: Runner, steps: int):
    """The same decode step issued the way a real model must (layer l+1's query does not exist before layer l
    is done): one lethe_decode_attend launch per layer, the launches replayed from a CUDA graph.  Returns
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
    r.step_no += 1 + 3 + steps                       # every replay appended one token per item
    ms = a.elapsed_time(b) / steps
    th = th0 + items * (3 + (steps + 1) / 2.0)       # mean length over the timed replays
    return ms, th


# ------------------------------------------------------------------------------------------- CPU baseline

def _sample_state(w, layers, seqs, max_steps, ratio):
    """The bounded sample of the workload the oracle is timed on: first `layers` layers, first `seqs` sequences."""
    ws = synth.shrink(w, n_layers=layers, batch=seqs)
    if w.page_tokens:                                    # ragged: the sample's sequences at their post-prune lengths, paged
        lens = torch.clamp((synth.ragged_lengths(w)[:seqs].double() * ratio).long(), min=w.k_min)
        cap = -(-(int(lens.max()) + max_steps + 8) // w.page_tokens) * w.page_tokens
        st = synth.initial_kv(ws, int(lens.max()), cap)
        st["len"][:] = lens[None, :, None].to(torch.int32)
        st = synth.to_paged(st, w.page_tokens, seed=w.seed)
        T = layers * lens
        return ws, st, cap, T, f"lengths {lens.tolist()} (= {ratio} of the sequences' lengths), 16-token pages"
    cap = w.mean_budget + max_steps + 8
    st = synth.initial_kv(ws, w.mean_budget, cap)
    T = torch.full((seqs,), layers * w.mean_budget, dtype=torch.int64)
    return ws, st, cap, T, f"~{w.mean_budget} tokens"


def _oracle_cache(oracle, ws, st, cap):
    seqs = st["len"].shape[1]
    if "page_table" in st:
        return oracle.OracleCache(ws.n_layers, seqs, ws.n_q_heads, ws.n_kv_heads, ws.head_dim, st["capacity_pages"],
                                  st["k"], st["v"], st["rel"], st["pos"], st["len"], ws.page_tokens, st["page_table"])
    return oracle.OracleCache(ws.n_layers, seqs, ws.n_q_heads, ws.n_kv_heads, ws.head_dim, cap, st["k"], st["v"],
                              st["rel"], st["pos"], st["len"])


def cpu_baseline(w, dev, seconds=12.0, layers=8, seqs=4, ratio=0.25):
    """The oracle, as it stands, on a bounded sample of the workload on the host cores."""
    import oracle
    threads = oracle.max_threads()
    oracle.set_threads(threads)
    layers = min(layers, w.n_layers)
    max_steps = 600
    ws, st, cap, T, what = _sample_state(w, layers, seqs, max_steps, ratio)
    oc = _oracle_cache(oracle, ws, st, cap)
    scale = synth.layer_scales(w)[:layers].contiguous()
    th = 0
    t0 = time.perf_counter()
    steps = 0
    while True:
        x = synth.step_inputs(ws, steps)
        s, *_ = oracle.decode_attend(oc, 0, layers, x["q"], x["k_new"], x["v_new"], x["token_pos"], scale, w.gamma)
        assert s == oracle.OK
        th += int(oc.len.sum())
        steps += 1
        if time.perf_counter() - t0 > seconds or steps >= max_steps - 90:
            break
    attend_s = time.perf_counter() - t0
    # one prune round on the sample, amortised like the GPU loop
    t1 = time.perf_counter()
    _, S = oracle.estimate_sparsity(oc)
    _, bud = oracle.alloc_budgets(S, T, w.k_min)
    oracle.rasr_prune(oc, bud, w.recent, w.sink)
    prune_s = time.perf_counter() - t1
    per_step = attend_s / steps + prune_s / w.prune_interval
    overlap = None
    if dev is not None:
        overlap = retained_set_overlap(w, ws, dev, oc, cap, steps, layers, seqs, scale, T, ratio)
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
            "sample": f"{layers} layers x {seqs} sequences x {w.n_kv_heads} KV heads at {what}, "
                      f"{steps} decode steps in {attend_s:.1f} s plus one prune round ({prune_s * 1e3:.0f} ms) "
                      f"amortised over {w.prune_interval} steps",
            "ms_per_sample_step": per_step * 1e3, "token_heads_per_sample_step": th / steps,
            "prune_round_ms_on_sample": prune_s * 1e3,
            "retained_set_overlap": overlap}


def retained_set_overlap(w, ws, dev, oc, cap, steps, layers, seqs, scale, T, ratio):
    """End-to-end agreement of what is kept: the GPU path replays the sample the oracle was just timed on (same
    initial cache, same per-step inputs, same number of steps, then one prune round), free-running on its own
    scores, and the retained positions of every item are compared with the oracle's."""
    from paper_2511_06029_b200 import binding
    _, st, _, _, _ = _sample_state(w, layers, seqs, 600, ratio)
    pt = st.get("page_table")
    gc = binding.Cache(ws.n_q_heads, *(st[k].to(dev) for k in ("k", "v", "rel", "pos", "len")),
                       None if pt is None else pt.to(dev))
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
        ctx.estimate_sparsity(gc, S)
        ctx.alloc_budgets(S, T.to(dev), w.k_min, bud)
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


# ------------------------------------------------------------------------------------------- config / arms

CONFIG_KEYS = ("workload", "global_batch", "l2", "parallelism", "resident_layers", "capacity", "variant", "splits",
               "launch_mode", "token_heads_per_step", "prune_rounds_timed", "prune_round_ms", "prune_round",
               "attend_ms_per_step", "attend_ms_median", "per_layer_launch", "segment_prune_8_segments",
               "collapsed_prune", "prefill_seed", "sweep", "note")


def workload_config(w, args, n_ranks, extra=None):
    """The `config` object; both arms print the same keys (None where a key does not apply to an arm)."""
    if w.page_tokens:
        shape = (f"{w.name}: L{w.n_layers} B{w.batch} Hq{w.n_q_heads}/Hkv{w.n_kv_heads} D{w.head_dim} bf16, "
                 f"{w.page_tokens}-token pages, per-sequence lengths uniform in [1024, 32768], budget ratio {args.ratio} of the "
                 f"length, recent {w.recent}, sink {w.sink}, prune every {w.prune_interval} steps, gamma {w.gamma}")
    else:
        shape = (f"{w.name}: L{w.n_layers} B{w.batch} Hq{w.n_q_heads}/Hkv{w.n_kv_heads} D{w.head_dim} bf16, "
                 f"mean budget {w.mean_budget}/layer, recent {w.recent}, sink {w.sink}, prune every "
                 f"{w.prune_interval} steps, gamma {w.gamma}")
    c = dict.fromkeys(CONFIG_KEYS)
    c.update({"workload": shape, "global_batch": w.batch * n_ranks,
              "l2": "inputs larger than L2 (every step streams more K/V than the 126 MB of L2)",
              "parallelism": f"dp{n_ranks} (sequences sharded, no data-path collective)"})
    if extra:
        c.update(extra)
    return c


def resolve_workload(args):
    """The workload the line is quoted on.  The ragged workload keeps one group of layers resident (the full state
    is 124 GB of K/V) and takes its prune interval / budget ratio from the command line."""
    w = synth.WORKLOADS[args.workload]
    if w.page_tokens:
        w = synth.shrink(w, n_layers=min(args.layers or RAGGED_RESIDENT_LAYERS, w.n_layers),
                         prune_interval=args.interval or w.prune_interval)
    elif args.layers:
        w = synth.shrink(w, n_layers=min(args.layers, w.n_layers))
    return w


def run_reference(args, w):
    """--impl reference: the oracle on the host cores, same metric / config keys.  Rank 0 alone works."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    base = cpu_baseline(w, None, seconds=max(5.0, min(60.0, 0.5 * (args.steps + args.warmup))), ratio=args.ratio)
    base.pop("retained_set_overlap", None)
    line = {"impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": base["ms_per_sample_step"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w, args, args.gpus, extra={
                "note": "oracle timed on a bounded sample per step",
                "resident_layers": w.n_layers if w.page_tokens else None}),
            "cpu_baseline": base,
            "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def launcher_selftest(args):
    """The multi-rank plumbing alone (no GPU work): every rank joins the process group the launcher set up,
    contributes a made-up (time, units) pair, and rank 0 prints what the reduction gives.  Used by the CPU tests."""
    import torch.distributed as dist
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        dev = torch.device("cpu")
        ids = dist_util.rank_batch_ids(rank, 4)
        (t,), (u, n, idsum) = dist_util.reduce_job(dist, dev, [10.0 + 5 * rank], [100.0 * (rank + 1), 1.0, float(ids.sum())])
        if rank == 0:
            print(json.dumps({"selftest": "launcher", "n_gpus": int(n), "max_ms": t, "units": u, "id_sum": idsum,
                              "value": dist_util.job_value(u, t)}))
        dist.barrier()
    finally:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------- sweep

def ragged_sweep(r: Runner, lens_seq, bytes_per_th, peak):
    """Budget-ratio x prune-interval sweep of the ragged workload.  Per point, from the un-pruned lengths n_b:
    (i) decode steps at n_b (the FullKV-like reference point), (ii) the prune round n_b -> floor(ratio n_b) with
    the three calls timed one by one, (iii) `interval` decode steps on the pruned cache; the amortised step is
    (iii) + (ii) / interval.  Before each point the cache is put back to n_b tokens per sequence (len, pos, rel = 0)
    and the relevance is warmed by attend-only steps; K / V values are random either way."""
    w, dev = r.w, r.dev
    L = w.n_layers
    stream = torch.cuda.current_stream(dev)
    ln0 = lens_seq.to(torch.int32).to(dev)[None, :, None].expand_as(r.cache.len).contiguous()
    pos0 = torch.arange(r.cache.cap_tokens, dtype=torch.int32, device=dev)
    items = r.cache.len.numel()
    points = []

    def timed(fn, n):
        a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(n):
            fn()
        b.record(stream)
        torch.cuda.synchronize(dev)
        return a.elapsed_time(b) / n

    full_ms = None
    for ratio in SWEEP_RATIOS:
        r.T = (L * torch.clamp((lens_seq.double() * ratio).long(), min=w.k_min)).to(dev)
        for interval in SWEEP_INTERVALS:
            r.cache.len.copy_(ln0); r.cache.pos.copy_(pos0.expand_as(r.cache.pos)); r.cache.rel.zero_()
            warm = min(interval, 64)
            for _ in range(warm):
                r.decode(append=False)
            th_full = int(r.cache.len.sum().item())
            if full_ms is None:                           # (i) is the same for every point: timed once
                full_ms = timed(lambda: r.decode(append=False), 3)
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            r.prune(events=ev)
            torch.cuda.synchronize(dev)
            pr = [ev[i].elapsed_time(ev[i + 1]) for i in range(3)]
            th_after = int(r.cache.len.sum().item())
            step_ms = timed(lambda: r.decode(), interval)
            r.check()
            th_mean = th_after + items * (interval + 1) / 2.0
            amort = step_ms + sum(pr) / interval
            points.append({"ratio": ratio, "interval": interval, "warm_steps": warm,
                           "token_heads_unpruned": th_full, "unpruned_step_ms": full_ms,
                           "unpruned_step_GBs": th_full * bytes_per_th / (full_ms * 1e-3) / 1e9,
                           "prune_round_us": sum(pr) * 1e3, "estimate_sparsity_us": pr[0] * 1e3,
                           "alloc_budgets_us": pr[1] * 1e3, "rasr_prune_us": pr[2] * 1e3,
                           "token_heads_after_prune": th_after, "pruned_step_ms": step_ms,
                           "pruned_step_GBs": th_mean * bytes_per_th / (step_ms * 1e-3) / 1e9,
                           "pruned_step_frac_of_peak": th_mean * bytes_per_th / (step_ms * 1e-3) / 1e9 / peak,
                           "amortised_step_ms": amort, "speedup_vs_unpruned": full_ms / amort})
    return points


# -------------------------------------------------------------------------------------------------- main

def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1024)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama8b", choices=["llama8b", "qwen7b", "longreason", "ragged"])
    ap.add_argument("--variant", type=int, default=0)
    ap.add_argument("--splits", type=int, default=0)
    ap.add_argument("--capacity", type=int, default=0)
    ap.add_argument("--layers", type=int, default=0, help="resident layers (ragged workload: default 7 of 28)")
    ap.add_argument("--ratio", type=float, default=0.25, help="ragged workload: budget as a fraction of each sequence's length")
    ap.add_argument("--interval", type=int, default=0, help="ragged workload: prune interval (default 256)")
    ap.add_argument("--sweep", action="store_true",
                    help="ragged workload: also run the budget-ratio x prune-interval sweep (config.sweep)")
    ap.add_argument("--prep-rounds", type=int, default=6,
                    help="untimed prune intervals run before warm-up so that lengths reach their budgets")
    ap.add_argument("--prune-rounds", type=int, default=3, help="prune rounds timed after the loop (at least 3)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-per-layer", action="store_true")
    ap.add_argument("--kv", choices=["bf16", "fp8", "fp8e5m2"], default="bf16",
                    help="storage of K and V: bf16 (the headline configuration), or e4m3 / e5m2 bytes with per-layer scales")
    ap.add_argument("--with-prefill", action="store_true",
                    help="also time lethe_prefill_seed on a prompt of the workload's length (informational)")
    ap.add_argument("--pl-variant", type=int, default=0, help="kernel variant of the per-layer launch mode")
    ap.add_argument("--pl-splits", type=int, default=0)
    ap.add_argument("--launcher-selftest", action="store_true", help=argparse.SUPPRESS)
    return ap.parse_args(argv)


def main():
    args = parse_args()
    launched = "WORLD_SIZE" in os.environ
    if args.gpus > 1 and not launched and (args.impl == "ours" or args.launcher_selftest):
        # no launcher around us: start the ranks ourselves, one process per GPU
        if not args.launcher_selftest:
            have = torch.cuda.device_count() if torch.cuda.is_available() else 0
            if have < args.gpus:
                raise SystemExit(f"bench.py --gpus {args.gpus}: only {have} CUDA device(s) visible; refusing to report "
                                 f"{args.gpus} GPUs from fewer")
        raise SystemExit(dist_util.spawn_ranks([sys.executable, os.path.abspath(__file__), *sys.argv[1:]], args.gpus))
    if args.launcher_selftest:
        launcher_selftest(args)
        return
    w = resolve_workload(args)
    if args.impl == "reference":
        run_reference(args, w)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != args.gpus:
        raise SystemExit(f"bench.py --gpus {args.gpus} was started with WORLD_SIZE={world}")
    if local >= torch.cuda.device_count():
        raise SystemExit(f"rank {rank}: no CUDA device {local}")
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
    peak, which = measured_peak()

    def prepare(capacity):
        """Runner brought to steady state (untimed): a few full prune intervals so that relevance, sparsity-driven
        budgets and lengths are those of a long trajectory (dense layers need several rounds to grow to their
        budget).  Returns the runner and the largest layer budget any of those rounds handed out."""
        r = Runner(w, dev, rank, capacity, args.variant, args.splits, kv=args.kv)
        largest = 0
        for _ in range(max(1, args.prep_rounds)):
            for _ in range(w.prune_interval):
                r.decode()
            r.prune()
            largest = max(largest, int(r.budgets.max().item()))   # budgets move from round to round with the relevance
            r.drift_if_due()
        r.check()
        return r, largest

    lens_seq = None
    if w.page_tokens:
        # Ragged: this rank's sequences at their drawn lengths n_b; steady state = floor(ratio n_b) tokens per layer
        # on average (never below the protected count), pruned back to that every interval.
        all_lens = synth.ragged_lengths(w, n=w.batch * world)
        lens_seq = all_lens[rank * w.batch:(rank + 1) * w.batch]
        capacity = -(-(int(all_lens.max()) + max(SWEEP_INTERVALS) + 2 * w.page_tokens) // w.page_tokens)   # pages per item
        T = w.n_layers * torch.clamp((lens_seq.double() * args.ratio).long(), min=w.k_min)
        r = Runner(w, dev, rank, capacity, args.variant, args.splits, kv=args.kv, lens_seq=lens_seq, total_budget=T)
        for _ in range(8):                               # relevance before the first round: a few attend-only steps
            r.decode(append=False)
        r.prune()
        for _ in range(max(1, min(args.prep_rounds, 2))):
            for _ in range(w.prune_interval):
                r.decode()
            r.prune()
        r.check()
        max_budget = int(r.budgets.max().item())
    elif args.capacity:
        # Capacity = largest layer budget + prune interval (+ slack), as a serving system would size it.  The budgets
        # follow from the measured sparsity, so a pilot run at a generous capacity finds them first.
        capacity = args.capacity
        r, max_budget = prepare(capacity)
    else:
        pilot, max_budget = prepare(3 * w.mean_budget)
        pilot.close()
        del pilot
        torch.cuda.empty_cache()
        capacity = -(-(max_budget + w.prune_interval + 32) // 64) * 64
        r, max_budget = prepare(capacity)
    if not w.page_tokens and max_budget + w.prune_interval > capacity:
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
    if not args.no_e2e:
        for _ in range(max(args.warmup, 3)):             # the host path's own warm-up (its first call sets up staging)
            r.decode(host=True)
            if r.prune_due():
                r.prune()
        barrier()
        e_total_ms, _, _, e_th = timed_loop(r, args.steps, host=True)
        barrier()
        r.check()
    th_per_launch = sum(th) / len(th)
    avg_attend_ms = sum(attend_ms) / len(attend_ms)
    # the prune round on its own clock, on every run (the timed loop holds one only when K crosses the interval)
    prune_round = time_prune_rounds(r, max(3, args.prune_rounds), bytes_per_th, avg_attend_ms, th_per_launch, peak)
    clocks = sampler.stop() if sampler else None
    per_layer = None
    if not args.no_per_layer and world == 1:
        room = w.prune_interval - (r.step_no % w.prune_interval)
        pl_steps = min(32, max(4, room - 8))
        r.ctx.set_tuning(args.pl_variant, args.pl_splits)
        r.ctx.set_tuning(51, 0)                          # layer pipelining: cached K / V tiles are fetched under the previous launch's tail
        ms_pl, th_pl = per_layer_mode(r, pl_steps)
        r.ctx.set_tuning(50, 0)
        r.ctx.set_tuning(args.variant, args.splits)
        r.check()
        gbs = th_pl * bytes_per_th / (ms_pl * 1e-3) / 1e9
        per_layer = {"ms_per_step": ms_pl, "token_heads_per_step": th_pl, "value": th_pl / (ms_pl * 1e-3),
                     "algorithmic_GBs": gbs, "frac": gbs / peak, "frac_of_8TBs_nominal": gbs / NOMINAL_HBM_GBS,
                     "mode": f"{w.n_layers} launches per step (one per layer), replayed from a CUDA graph, "
                             f"{pl_steps} steps; layer pipelining on (a launch fetches cached K / V tiles before the "
                             f"previous launch has completed, and reads its query only after it has); not part of `value`"}

    sweep = None
    if args.sweep and w.page_tokens and world == 1:
        sweep = ragged_sweep(r, lens_seq, bytes_per_th, peak)

    # Retention by the collapsed score of Eq. 2 (one set per sequence), timed once on the live state with the
    # budgets a RASR round would get now: the row traffic of such a round.  Only the heads' lengths are aligned here (the
    # earlier rounds pruned head by head), so this is a timing of the call, not a meaningful retention.
    collapsed = None
    if not args.no_per_layer and world == 1 and not w.page_tokens:
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
    if not args.no_per_layer and world == 1 and not w.page_tokens:
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
    if args.with_prefill and world == 1 and not w.page_tokens:
        prefill = time_prefill(r, w, dev)
    e_ms = e_total_ms if not args.no_e2e else 0.0
    e_u = float(sum(e_th)) if not args.no_e2e else 0.0
    (t_ms, e_total_ms), (units, e_units, n_ranks) = dist_util.reduce_job(dist, dev, [total_ms, e_ms],
                                                                        [float(sum(th)), e_u, 1.0])
    n_ranks = int(round(n_ranks))

    if rank == 0:
        achieved = th_per_launch * bytes_per_th / (avg_attend_ms * 1e-3) / 1e9
        B_r = w.batch
        h2d = (w.n_layers * B_r * (w.n_q_heads + 2 * w.n_kv_heads) * w.head_dim * 2 + B_r * 4)
        d2h = w.n_layers * B_r * w.n_q_heads * w.head_dim * 2
        traffic = NCU_TRAFFIC.get(args.workload if args.kv == "bf16" else f"{args.workload}:{args.kv}") if args.variant == 0 else None
        line = {
            "metric": METRIC, "value": dist_util.job_value(units, t_ms), "unit": UNIT, "n_gpus": n_ranks, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": t_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if args.kv == "bf16" else
                     f"fp8 K/V ({'e4m3' if args.kv == 'fp8' else 'e5m2'} bytes, per-layer scales), bf16 activations, 8-bit tensor-core products (queries and probabilities as three e4m3 terms), fp32 accumulation",
            "data": "synthetic",
            "config": workload_config(w, args, n_ranks, extra={
                "resident_layers": w.n_layers if w.page_tokens else None,
                "capacity": capacity, "variant": args.variant, "splits": args.splits,
                "launch_mode": "all resident layers in one lethe_decode_attend call per step",
                "token_heads_per_step": th_per_launch,
                "prune_rounds_timed": prune_round["rounds_timed"],
                "prune_round_ms": prune_round["prune_round_us"] * 1e-3,
                "prune_round": dict(prune_round, rounds_inside_the_timed_loop=len(prune_ms),
                                    ms_inside_the_timed_loop=(sum(prune_ms) / len(prune_ms)) if prune_ms else None),
                "attend_ms_per_step": avg_attend_ms,
                "attend_ms_median": statistics.median(attend_ms),
                "per_layer_launch": per_layer,
                "segment_prune_8_segments": segment,
                "collapsed_prune": collapsed,
                "prefill_seed": prefill,
                "sweep": sweep}),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "peak_source": f"of {which}", "frac_of_8TBs_nominal": achieved / NOMINAL_HBM_GBS,
                         "kernel": "attend (dominant kernel; one launch per step)",
                         "traffic": traffic[0] * th_per_launch if traffic else None,
                         "traffic_source": (f"not measured in this run: {traffic[0]} B per token-head from the ncu capture "
                                            f"summarised in {traffic[1]}, scaled to this launch's token-heads") if traffic else None,
                         "with_amortised_prune": prune_round["decode_attend_plus_amortised_prune"]},
            "gpu_launches": launches, "clocks": clocks,
        }
        if not args.no_e2e:
            line["e2e"] = {"value": dist_util.job_value(e_units, e_total_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
                           "d2h_bytes_per_step": d2h, "ms_per_step": e_total_ms / args.steps,
                           "transfer": "pinned host buffers; the attend kernel reads the step's inputs from them and "
                                       "writes out into them over the bus, inside the timed launch (pageable buffers "
                                       "would take staged copies)"}
        if not args.no_cpu_baseline and world == 1:   # the oracle is timed beside the single-GPU run only
            line["cpu_baseline"] = cpu_baseline(w, dev, ratio=args.ratio)
            line["retained_set_overlap"] = line["cpu_baseline"].pop("retained_set_overlap", None)
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def time_prefill(r, w, dev):
    """lethe_prefill_seed on a prompt of the workload's length, both engines (informational)."""
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
    return {"prompt_len": P, "engines": engines, "bound": "alu (ex2: one exponential per logit and pass)",
            "ex2_peak_per_s": xu_peak,
            "note": "two passes (statistics, column sums), 2 launches per call; tcgen05 = default engine "
                    "(accumulators in tensor memory, TMA operand tiles), mma_sync = the legacy tensor path"}


if __name__ == "__main__":
    main()
