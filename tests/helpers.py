"""Small helpers shared by the tests (state construction and the decode/prune loop around the oracle)."""
import torch

import oracle


def random_cache(L, B, Hq, Hkv, D, cap, lens, dtype=torch.float32, seed=0, rel_init="zero"):
    """OracleCache with Gaussian K/V; lens: int or tensor [L][B][Hkv]."""
    g = torch.Generator().manual_seed(seed)
    k = torch.randn((L, B, Hkv, cap, D), generator=g).to(dtype)
    v = torch.randn((L, B, Hkv, cap, D), generator=g).to(dtype)
    if rel_init == "zero":
        rel = torch.zeros((L, B, Hkv, cap), dtype=torch.float32)
    else:
        rel = torch.rand((L, B, Hkv, cap), generator=g, dtype=torch.float32)
    pos = torch.arange(cap, dtype=torch.int32).expand(L, B, Hkv, cap).contiguous()
    if isinstance(lens, int):
        ln = torch.full((L, B, Hkv), lens, dtype=torch.int32)
    else:
        ln = lens.to(torch.int32).contiguous()
    return oracle.OracleCache(L, B, Hq, Hkv, D, cap, k, v, rel, pos, ln)


def cache_from_state(w, state, capacity):
    """OracleCache over the tensors of a synth state dict (contiguous or paged)."""
    if "page_table" in state:
        return oracle.OracleCache(w.n_layers, state["len"].shape[1], w.n_q_heads, w.n_kv_heads, w.head_dim,
                                  state["capacity_pages"], state["k"], state["v"], state["rel"], state["pos"],
                                  state["len"], w.page_tokens, state["page_table"])
    return oracle.OracleCache(w.n_layers, state["len"].shape[1], w.n_q_heads, w.n_kv_heads, w.head_dim,
                              capacity, state["k"], state["v"], state["rel"], state["pos"], state["len"])


def oracle_prune_round(cache, total_budget, k_min, recent, sink, max_k=0):
    """Sparsity -> budgets -> retention on the oracle (the prune round of Sec. 4.1-4.3)."""
    st, S = oracle.estimate_sparsity(cache)
    assert st == oracle.OK
    st, budgets = oracle.alloc_budgets(S, total_budget, k_min)
    assert st == oracle.OK
    st, keep = oracle.rasr_prune(cache, budgets, recent, sink, max_k=max_k)
    return st, S, budgets, keep
