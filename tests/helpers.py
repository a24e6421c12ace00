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


# ----------------------------------------------------------------------------- GPU side (tests marked gpu)

def gpu_context():
    """Build (if stale) and load the CUDA library, return a Context on cuda:0."""
    from paper_2511_06029_b200 import binding, build
    build.build()
    return binding.Context(0)


def to_device(oc):
    """Upload an OracleCache to the GPU as a binding.Cache (deep copy)."""
    from paper_2511_06029_b200 import binding
    dev = torch.device("cuda", 0)
    pt = None if oc.page_table is None else oc.page_table.to(dev)
    return binding.Cache(oc.n_q_heads, oc.k.to(dev), oc.v.to(dev), oc.rel.to(dev), oc.pos.to(dev), oc.len.to(dev), pt,
                         k_scale=oc.k_scale, v_scale=oc.v_scale)


def sync_state(gc, oc):
    """Overwrite the GPU cache state with the oracle's (call-by-call parity: identical inputs for the next call)."""
    gc.k.view(torch.uint8).copy_(oc.k.view(torch.uint8)); gc.v.view(torch.uint8).copy_(oc.v.view(torch.uint8))
    gc.rel.copy_(oc.rel); gc.pos.copy_(oc.pos); gc.len.copy_(oc.len)


def logical_rows(k, v, rel, pos, ln, page_table=None, page_tokens=0):
    """Per item (K rows, V rows, rel, pos) of the first len slots, as CPU tensors, for either layout."""
    k, v, rel, pos, ln = k.cpu(), v.cpu(), rel.cpu(), pos.cpu(), ln.cpu()
    if k.dtype in (torch.float8_e4m3fn, torch.float8_e5m2):   # compare quantised rows as the bytes they are
        k, v = k.view(torch.uint8), v.view(torch.uint8)
    L, B, H = ln.shape
    out = []
    for l in range(L):
        for b in range(B):
            for h in range(H):
                n = int(ln[l, b, h])
                if page_table is not None:
                    pg = page_table.cpu()[l, b, h].long()
                    kk = k[pg].reshape(-1, k.shape[-1])[:n]; vv = v[pg].reshape(-1, v.shape[-1])[:n]
                else:
                    kk = k[l, b, h, :n]; vv = v[l, b, h, :n]
                out.append((kk, vv, rel[l, b, h, :n], pos[l, b, h, :n]))
    return out


def assert_state_matches(gc, oc, rel_rtol=1e-3, rel_atol=1e-6, exact_rel=False):
    """len, pos, K, V rows bit-exact; rel within tolerance (or bit-exact after a prune on identical scores)."""
    assert torch.equal(gc.len.cpu(), oc.len)
    g = logical_rows(gc.k, gc.v, gc.rel, gc.pos, gc.len, gc.page_table, gc.page_tokens)
    o = logical_rows(oc.k, oc.v, oc.rel, oc.pos, oc.len, oc.page_table, oc.page_tokens)
    for i, ((gk, gv, gr, gp), (ok, ov, orl, op)) in enumerate(zip(g, o)):
        assert torch.equal(gk.view(torch.uint8), ok.view(torch.uint8)), f"K rows differ at item {i}"
        assert torch.equal(gv.view(torch.uint8), ov.view(torch.uint8)), f"V rows differ at item {i}"
        assert torch.equal(gp, op), f"pos differs at item {i}"
        if exact_rel:
            assert torch.equal(gr, orl), f"rel differs at item {i}"
        else:
            assert torch.allclose(gr, orl, rtol=rel_rtol, atol=rel_atol), \
                f"rel differs at item {i}: max abs {float((gr - orl).abs().max())}"
