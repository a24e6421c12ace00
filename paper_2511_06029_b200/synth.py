"""Seeded synthetic workloads for the Lethe hot path.

This module only *draws inputs*: cache contents, per-step q / k_new / v_new,
per-layer softmax scales and the workload table.  It contains none of the
method's arithmetic (no softmax, no relevance, no selection), so the CUDA
binding, the CPU oracle's tests and the benchmark can all use it without
sharing anything that is being verified.

The five workloads mirror the shapes of the paper's evaluation (decode-dominated
chain-of-thought generation on GQA Llama/Qwen geometries, Sec. 5.1) with
synthetic values: Gaussian q/K/V plus a small set of "anchor" tokens whose keys
are scaled up so that attention is sparse, and layer-dependent temperature or
anchor density so that sparsity differs across layers (Sec. 3.2).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Dict, Optional

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: torch.dtype
    prompt_len: int          # KV length before the first decode step
    gen_steps: int           # decode steps of the full trajectory
    mean_budget: int         # mean retained tokens per layer (global budget = n_layers * mean_budget)
    recent: int              # recent window r (Algorithm 1)
    sink: int                # sink length s_len (Algorithm 1)
    prune_interval: int
    gamma: float             # decay of Eq. 5
    seed: int
    anchor_rule: str         # "fixed16" | "per_seq" | "per_layer_beta"
    anchor_gain: float
    anchor_density: float = 0.01
    temp_range: Optional[tuple] = None   # per-layer attention temperature ~ U[a, b]
    drift_period: int = 0                # re-draw the anchor set every this many decode steps (0 = never)
    page_tokens: int = 0                 # > 0: paged KV layout

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def total_budget(self) -> int:
        return self.n_layers * self.mean_budget

    @property
    def k_min(self) -> int:
        return self.recent + self.sink


WORKLOADS: Dict[str, Workload] = {
    "tiny": Workload("tiny", 1, 1, 8, 2, 64, torch.float32, 512, 64, 128, 32, 4, 16, 0.99, 0,
                     "fixed16", 4.0),
    "llama8b": Workload("llama8b", 32, 8, 32, 8, 128, torch.bfloat16, 512, 4096, 1024, 64, 4, 128, 0.99, 1,
                        "per_seq", 3.0, temp_range=(0.5, 2.0)),
    "qwen7b": Workload("qwen7b", 28, 32, 28, 4, 128, torch.bfloat16, 256, 16384, 2048, 128, 4, 256, 0.99, 2,
                       "per_layer_beta", 3.0),
    "longreason": Workload("longreason", 32, 64, 32, 8, 128, torch.bfloat16, 1024, 32768, 2048, 128, 4, 512,
                           0.99, 3, "per_seq", 3.0, temp_range=(0.5, 2.0), drift_period=2048),
    "ragged": Workload("ragged", 28, 128, 28, 4, 128, torch.bfloat16, 1024, 0, 2048, 128, 4, 256, 0.99, 4,
                       "per_layer_beta", 3.0, page_tokens=16),
}


def shrink(w: Workload, **kw) -> Workload:
    """Same workload with some fields replaced (e.g. a smaller batch for a CPU-sized parity case)."""
    return replace(w, **kw)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) & 0x7FFFFFFFFFFFFFFF)
    return g


def _mix64(x: torch.Tensor) -> torch.Tensor:
    """Stateless 64-bit integer mixer (splitmix-style) on int64 tensors; identical on CPU and GPU."""
    x = x * -7046029254386353131          # 0x9E3779B97F4A7C15 as signed
    x = (x ^ ((x >> 30) & 0x3FFFFFFFF)) * -4658895280553007687   # 0xBF58476D1CE4E5B9
    x = (x ^ ((x >> 27) & 0x1FFFFFFFFF)) * -7723592293110705685  # 0x94D049BB133111EB
    return x ^ ((x >> 31) & 0x1FFFFFFFF)


def layer_scales(w: Workload) -> torch.Tensor:
    """Per-layer softmax scale 1/(sqrt(D) * T_l); T_l = 1 unless the workload draws temperatures."""
    base = 1.0 / math.sqrt(w.head_dim)
    if w.temp_range is None:
        return torch.full((w.n_layers,), base, dtype=torch.float32)
    g = _gen(w.seed * 7919 + 11, "cpu")
    a, b = w.temp_range
    t = a + (b - a) * torch.rand(w.n_layers, generator=g, dtype=torch.float64)
    return (base / t).to(torch.float32)


def layer_anchor_density(w: Workload) -> torch.Tensor:
    """Anchor density per layer: constant, or Beta(0.5, 5) per layer."""
    if w.anchor_rule == "per_layer_beta":
        torch.manual_seed(w.seed * 104729 + 5)
        return torch.distributions.Beta(torch.tensor(0.5, dtype=torch.float64),
                                        torch.tensor(5.0, dtype=torch.float64)).sample((w.n_layers,))
    return torch.full((w.n_layers,), w.anchor_density, dtype=torch.float64)


def drift_epoch(w: Workload, step: int) -> int:
    """Epoch of the anchor draw that is in force at decode step `step` (0 while the workload does not drift)."""
    return step // w.drift_period if w.drift_period > 0 else 0


def _anchor_hit(w: Workload, lay: torch.Tensor, bid: torch.Tensor, pos: torch.Tensor, epoch: int) -> torch.Tensor:
    """Elementwise anchor test on broadcastable int64 tensors (layer, global sequence id, original position)."""
    if w.anchor_rule == "per_seq":
        lay = torch.zeros_like(lay)           # shared across layers
    key = (w.seed + 1) * 1000003 + lay * 7368787 + bid * 15485863 + pos * 2654435761 + int(epoch) * 40503
    u = (_mix64(key) & 0xFFFFFF).to(torch.float64) / float(1 << 24)
    dens = layer_anchor_density(w).to(pos.device)
    return u < dens[lay]


def anchor_flags(w: Workload, positions: torch.Tensor, batch_ids: torch.Tensor, epoch: int = 0) -> torch.Tensor:
    """bool [L][len(batch_ids)][len(positions)]: is the token at an original position an anchor during `epoch`?

    Counter-based (a hash of seed, layer or 0, sequence, position, epoch), so any position can be queried on any
    device at any time with the same answer.  A drifting workload re-draws the whole set every `drift_period`
    decode steps: the draws of different epochs are independent, old tokens included.
    """
    dev = positions.device
    pos = positions.to(torch.int64)
    bid = batch_ids.to(torch.int64).to(dev)
    L = w.n_layers
    if w.anchor_rule == "fixed16":
        g = _gen(w.seed * 31 + 3, "cpu")
        chosen = torch.randperm(w.prompt_len, generator=g)[:16].to(dev)
        hit = (pos[:, None] == chosen[None, :]).any(dim=1)
        return hit[None, None, :].expand(L, bid.numel(), pos.numel()).clone()
    lay = torch.arange(L, device=dev, dtype=torch.int64)
    return _anchor_hit(w, lay[:, None, None], bid[None, :, None], pos[None, None, :], epoch)


def apply_drift(w: Workload, k: torch.Tensor, pos: torch.Tensor, batch_ids: torch.Tensor, old_epoch: int,
                new_epoch: int) -> None:
    """Re-draw the anchors of a contiguous cache in place: K rows [L][B][Hkv][cap][D] of tokens that stop being
    anchors are divided by the anchor gain, rows of tokens that become anchors are multiplied by it (fp32
    arithmetic, one rounding to the cache dtype); `pos` [L][B][Hkv][cap] says which token sits in each slot.
    Harness work between decode steps (an epoch boundary), not part of the method."""
    if old_epoch == new_epoch or w.anchor_rule == "fixed16":
        return
    L, B = k.shape[0], k.shape[1]
    lay = torch.arange(L, device=k.device, dtype=torch.int64)[:, None, None]
    for b in range(B):
        bid = batch_ids[b].to(torch.int64).to(k.device)
        p = pos[:, b].to(torch.int64)                                       # [L][Hkv][cap]
        f_old = _anchor_hit(w, lay, bid, p, old_epoch)
        f_new = _anchor_hit(w, lay, bid, p, new_epoch)
        factor = torch.ones(p.shape, dtype=torch.float32, device=k.device)
        factor[f_new & ~f_old] = float(w.anchor_gain)
        factor[f_old & ~f_new] = 1.0 / float(w.anchor_gain)
        k[:, b] = (k[:, b].to(torch.float32) * factor[..., None]).to(k.dtype)


def _randn(shape, g: torch.Generator, dtype: torch.dtype, device) -> torch.Tensor:
    return torch.randn(shape, generator=g, dtype=torch.float32, device=device)


def initial_kv(w: Workload, n0: int, capacity: int, device="cpu", batch_ids: Optional[torch.Tensor] = None,
               layer_chunk: int = 4):
    """Contiguous cache state holding n0 tokens per item: dict(k, v, rel, pos, len).

    K, V ~ N(0,1) rounded to the workload dtype; anchor rows of K are multiplied by the anchor gain (in
    fp32, then rounded).  rel = 0, pos = 0..n0-1.
    """
    if batch_ids is None:
        batch_ids = torch.arange(w.batch)
    B = int(batch_ids.numel())
    L, H, D = w.n_layers, w.n_kv_heads, w.head_dim
    k = torch.zeros((L, B, H, capacity, D), dtype=w.dtype, device=device)
    v = torch.zeros((L, B, H, capacity, D), dtype=w.dtype, device=device)
    g = _gen(w.seed * 1315423911 + 17, device)
    positions = torch.arange(n0, device=device)
    flags = anchor_flags(w, positions, batch_ids)          # [L][B][n0]
    for l0 in range(0, L, layer_chunk):
        l1 = min(L, l0 + layer_chunk)
        kk = _randn((l1 - l0, B, H, n0, D), g, w.dtype, device)
        gain = torch.where(flags[l0:l1], w.anchor_gain, 1.0).to(torch.float32)
        kk = kk * gain[:, :, None, :, None]
        k[l0:l1, :, :, :n0] = kk.to(w.dtype)
        v[l0:l1, :, :, :n0] = _randn((l1 - l0, B, H, n0, D), g, w.dtype, device).to(w.dtype)
    rel = torch.zeros((L, B, H, capacity), dtype=torch.float32, device=device)
    pos = torch.zeros((L, B, H, capacity), dtype=torch.int32, device=device)
    pos[..., :n0] = positions.to(torch.int32)
    ln = torch.full((L, B, H), n0, dtype=torch.int32, device=device)
    return {"k": k, "v": v, "rel": rel, "pos": pos, "len": ln}


def step_inputs(w: Workload, step: int, device="cpu", batch_ids: Optional[torch.Tensor] = None):
    """Inputs of decode step `step` (0-based): dict(q, k_new, v_new, token_pos).

    q [L][B][Hq][D], k_new / v_new [L][B][Hkv][D] in the workload dtype, token_pos [B] int32 = prompt_len +
    step.  The generated token's key is an anchor by the same rule as the cache (never for "fixed16").
    """
    if batch_ids is None:
        batch_ids = torch.arange(w.batch)
    B = int(batch_ids.numel())
    L, Hq, H, D = w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim
    g = _gen((w.seed * 2654435761 + 1013904223 * (step + 1)) % (1 << 62), device)
    q = _randn((L, B, Hq, D), g, w.dtype, device)
    kn = _randn((L, B, H, D), g, w.dtype, device)
    vn = _randn((L, B, H, D), g, w.dtype, device)
    p = w.prompt_len + step
    if w.anchor_rule != "fixed16":
        fl = anchor_flags(w, torch.tensor([p], device=device), batch_ids, drift_epoch(w, step))       # [L][B][1]
        kn = kn * torch.where(fl, w.anchor_gain, 1.0).to(torch.float32)[:, :, :, None]
    token_pos = torch.full((B,), p, dtype=torch.int32, device=device)
    return {"q": q.to(w.dtype), "k_new": kn.to(w.dtype), "v_new": vn.to(w.dtype), "token_pos": token_pos}


def ragged_lengths(w: Workload, lo: int = 1024, hi: int = 32768, n: Optional[int] = None) -> torch.Tensor:
    """Per-sequence KV length, uniform integer in [lo, hi] (ragged-batch workload), for the global sequences
    0..n-1 (default: the workload's batch).  A longer draw starts with the shorter one, so ranks that hold
    different slices of one job agree on every sequence's length."""
    g = _gen(w.seed * 48271 + 9, "cpu")
    return torch.randint(lo, hi + 1, (n or w.batch,), generator=g, dtype=torch.int64)


def to_paged(state: dict, page_tokens: int, seed: int, spare_pages: int = 0):
    """Re-store a contiguous state in `page_tokens`-token pages with a shuffled (fragmented) page table.

    Returns dict(k, v, rel, pos, len, page_table, capacity_pages): k/v are pools [n_pages][page_tokens][D];
    page_table is [L][B][Hkv][capacity_pages] int32.  The contiguous capacity must be a multiple of page_tokens.
    """
    k, v = state["k"], state["v"]
    L, B, H, cap, D = k.shape
    assert cap % page_tokens == 0
    cp = cap // page_tokens
    n_pages = L * B * H * cp + spare_pages
    g = _gen(seed * 69621 + 23, "cpu")
    perm = torch.randperm(n_pages, generator=g)[: L * B * H * cp].to(k.device)
    table = perm.reshape(L, B, H, cp).to(torch.int32)
    kp = torch.zeros((n_pages, page_tokens, D), dtype=k.dtype, device=k.device)
    vp = torch.zeros((n_pages, page_tokens, D), dtype=k.dtype, device=k.device)
    kp[perm] = k.reshape(L * B * H * cp, page_tokens, D)
    vp[perm] = v.reshape(L * B * H * cp, page_tokens, D)
    return {"k": kp, "v": vp, "rel": state["rel"].clone(), "pos": state["pos"].clone(), "len": state["len"].clone(),
            "page_table": table, "capacity_pages": cp}
