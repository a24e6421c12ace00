"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element, on the same
seeded inputs.  Tolerances: integer / index / moved-row results bit-exact; attention output max-abs 2e-2 for
bf16 caches and 1e-4 for fp32; relevance and sparsity |d| <= 1e-3 |ref| + 1e-6.
"""
import pytest
import torch

import oracle
from helpers import (assert_state_matches, cache_from_state, gpu_context, oracle_prune_round, random_cache, sync_state,
                     to_device)
from paper_2511_06029_b200 import synth

pytestmark = pytest.mark.gpu

OUT_TOL = {torch.float32: 1e-4, torch.bfloat16: 2e-2}


@pytest.fixture(scope="module")
def ctx():
    c = gpu_context()
    yield c
    c.close()


def _lens(L, B, Hkv, cap, seed, special=()):
    g = torch.Generator().manual_seed(seed)
    ln = torch.randint(1, cap, (L, B, Hkv), generator=g)
    flat = ln.view(-1)
    for i, val in enumerate(special):
        flat[i % flat.numel()] = val
    return ln


def _step(ctx, oc, gc, q, kn, vn, tp, scale, gamma, l0, l1, want_lse=True):
    """Run one decode call on both sides and compare everything it produces."""
    dev = gc.device
    st, o_out, o_lse, _ = oracle.decode_attend(oc, l0, l1, q, kn, vn, tp, scale, gamma, want_lse=True)
    assert st == oracle.OK
    out = torch.full_like(q, float("nan"), device=dev)
    lse = torch.full((l1 - l0, oc.batch, oc.n_q_heads), float("nan"), device=dev) if want_lse else None
    ctx.decode_attend(gc, l0, l1, q.to(dev), None if kn is None else kn.to(dev), None if vn is None else vn.to(dev),
                      None if tp is None else tp.to(dev), scale.tolist(), gamma, out, lse)
    st, item = ctx.poll_status()
    assert st == 0, (st, item)
    tol = OUT_TOL[q.dtype]
    err = (out.cpu().double() - o_out.double()).abs().max().item()
    assert err <= tol, f"out max-abs error {err}"
    if want_lse:
        fin = torch.isfinite(o_lse)
        assert torch.equal(torch.isfinite(lse.cpu()), fin)
        assert torch.allclose(lse.cpu()[fin], o_lse[fin], rtol=1e-4, atol=1e-4)
    assert_state_matches(gc, oc)
    return out


CASES = [
    # dtype, D, Hq, Hkv, cap, variant, splits
    (torch.float32, 64, 8, 2, 200, 1, 1),
    (torch.float32, 64, 8, 2, 200, 1, 4),
    (torch.float32, 128, 4, 4, 150, 1, 2),
    (torch.bfloat16, 128, 32, 8, 300, 1, 1),
    (torch.bfloat16, 64, 14, 2, 300, 1, 8),
    (torch.bfloat16, 128, 32, 8, 300, 2, 1),
    (torch.bfloat16, 128, 32, 8, 300, 2, 2),
    (torch.bfloat16, 128, 28, 4, 300, 2, 4),
    (torch.bfloat16, 128, 28, 4, 700, 3, 1),
    (torch.bfloat16, 128, 8, 1, 700, 3, 8),
    (torch.bfloat16, 128, 6, 2, 1000, 3, 16),
    (torch.bfloat16, 64, 8, 2, 300, 2, 2),
    (torch.bfloat16, 64, 10, 2, 500, 3, 4),
    (torch.bfloat16, 128, 32, 8, 300, 4, 2),
    (torch.bfloat16, 128, 28, 4, 300, 5, 4),
    (torch.bfloat16, 64, 8, 2, 300, 6, 1),
    (torch.bfloat16, 128, 8, 2, 300, 7, 2),
    (torch.bfloat16, 128, 32, 8, 300, 8, 0),
    (torch.bfloat16, 128, 28, 4, 700, 9, 1),
    (torch.bfloat16, 64, 14, 2, 300, 10, 0),
    (torch.bfloat16, 128, 4, 1, 300, 11, 0),
    (torch.bfloat16, 64, 16, 2, 500, 12, 0),
    (torch.bfloat16, 128, 6, 2, 300, 13, 0),
    (torch.bfloat16, 128, 32, 8, 300, 16, 0),
    (torch.bfloat16, 128, 28, 4, 700, 17, 1),
    (torch.bfloat16, 64, 14, 2, 300, 18, 0),
    (torch.bfloat16, 128, 4, 1, 300, 19, 0),
    (torch.bfloat16, 64, 16, 2, 500, 20, 0),
    (torch.bfloat16, 128, 6, 2, 300, 21, 0),
    (torch.bfloat16, 128, 32, 8, 300, 24, 0),
    (torch.bfloat16, 128, 28, 4, 700, 26, 0),
    (torch.bfloat16, 64, 14, 2, 300, 27, 0),
    (torch.bfloat16, 64, 16, 2, 500, 29, 0),
    (torch.bfloat16, 128, 32, 8, 300, 32, 0),
    (torch.bfloat16, 128, 28, 4, 700, 33, 3),
    (torch.bfloat16, 64, 14, 2, 300, 34, 5),
    (torch.bfloat16, 128, 8, 1, 1000, 35, 16),
    (torch.bfloat16, 64, 16, 2, 500, 36, 1),
    (torch.bfloat16, 128, 6, 2, 300, 37, 7),
    (torch.bfloat16, 128, 32, 8, 300, 44, 1),
    (torch.bfloat16, 128, 32, 8, 300, 44, 2),
    (torch.bfloat16, 128, 28, 4, 300, 44, 4),
    (torch.bfloat16, 128, 28, 4, 700, 45, 1),
    (torch.bfloat16, 128, 8, 1, 700, 45, 8),
    (torch.bfloat16, 128, 6, 2, 1000, 45, 16),
    (torch.bfloat16, 64, 8, 2, 300, 46, 2),
    (torch.bfloat16, 128, 28, 4, 700, 46, 4),            # seven query heads per KV head: the instance with the group size compiled in
    (torch.bfloat16, 128, 28, 4, 300, 8, 0),             # the same for the persistent kernel's automatic shape
    (torch.bfloat16, 128, 40, 8, 300, 16, 0),            # five and eight heads per KV head: the asynchronous kernel's compiled-in sizes
    (torch.bfloat16, 128, 64, 8, 300, 16, 0),
    (torch.bfloat16, 64, 10, 2, 500, 47, 4),
    (torch.bfloat16, 128, 32, 8, 300, 48, 0),
    (torch.bfloat16, 64, 16, 2, 300, 49, 2),
    (torch.bfloat16, 128, 8, 8, 260, 0, 0),
    (torch.float32, 128, 16, 2, 260, 0, 0),
]


@pytest.mark.parametrize("dtype,D,Hq,Hkv,cap,variant,splits", CASES)
def test_decode_attend_parity(ctx, dtype, D, Hq, Hkv, cap, variant, splits):
    """Ragged lengths spanning several 16-token groups and ragged tails; append and attend-only steps; a layer
    sub-range; every kernel variant and cluster size."""
    L, B = 3, 2
    lens = _lens(L, B, Hkv, cap - 4, seed=cap + D, special=(1, 15, 16, 17, cap - 5, 33))
    oc = random_cache(L, B, Hq, Hkv, D, cap, lens, dtype=dtype, seed=D + Hq, rel_init="rand")
    gc = to_device(oc)
    ctx.set_tuning(variant, splits)
    try:
        g = torch.Generator().manual_seed(99)
        scale = torch.tensor([0.09, 0.2, 0.05], dtype=torch.float32) * (128 / D) ** 0.5
        for step, (l0, l1, app) in enumerate([(0, 3, True), (1, 2, False), (0, 3, True), (2, 3, True)]):
            nl = l1 - l0
            q = torch.randn((nl, B, Hq, D), generator=g).to(dtype)
            kn = torch.randn((nl, B, Hkv, D), generator=g).to(dtype) if app else None
            vn = torch.randn((nl, B, Hkv, D), generator=g).to(dtype) if app else None
            tp = torch.tensor([1000 + step, 2000 + step], dtype=torch.int32) if app else None
            _step(ctx, oc, gc, q, kn, vn, tp, scale, 0.9, l0, l1)
    finally:
        ctx.set_tuning(0, 0)


@pytest.mark.parametrize("variant", [8, 9, 10, 12, 13, 16, 17, 18, 19, 21, 24, 26, 27, 29])
def test_persistent_queue_many_items(ctx, variant):
    """More items than SMs, so every CTA of the persistent kernel walks several items through its queue and
    prefetches across item boundaries; lengths from 0 to several hundred, including tiny items that leave
    some warps without work, and one full item."""
    from paper_2511_06029_b200 import binding
    L, B, Hq, Hkv, D, cap = 5, 8, 16, 8, 128, 400
    lens = _lens(L, B, Hkv, cap - 6, seed=variant, special=(1, 2, 15, 16, 17, 31, 32, 33, 47, 48, 49, 127, 128, 129,
                                                           255, 256, 257, 390))
    oc = random_cache(L, B, Hq, Hkv, D, cap, lens, dtype=torch.bfloat16, seed=variant, rel_init="rand")
    gc = to_device(oc)
    ctx.set_tuning(variant, 0)
    try:
        g = torch.Generator().manual_seed(5)
        scale = torch.tensor([0.09, 0.2, 0.05, 0.12, 0.07], dtype=torch.float32)
        for step in range(4):
            app = step != 1
            q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
            kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16) if app else None
            vn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16) if app else None
            tp = torch.arange(B, dtype=torch.int32) + 1000 * step if app else None
            _step(ctx, oc, gc, q, kn, vn, tp, scale, 0.97, 0, L)
        # an empty item and a full one in the same launch
        oc.len[2, 3, 4] = 0; oc.len[4, 7, 7] = cap
        sync_state(gc, oc)
        q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
        _step(ctx, oc, gc, q, None, None, None, scale, 0.97, 0, L)            # attend only: empty item -> zeros, -inf
        kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16).cuda()
        out = torch.full((L, B, Hq, D), 7.0, dtype=torch.bfloat16, device="cuda")
        before_k = gc.k[4, 7, 7].clone(); before_rel = gc.rel[4, 7, 7].clone()
        ctx.decode_attend(gc, 0, L, q.cuda(), kn, kn, torch.zeros(B, dtype=torch.int32).cuda(), scale.tolist(), 0.97, out)
        st, item = ctx.poll_status()
        assert st == binding.ERR_CAPACITY and item == (4 * B + 7) * Hkv + 7
        assert int(gc.len[4, 7, 7]) == cap and int(gc.len[2, 3, 4]) == 1
        assert torch.equal(gc.k[4, 7, 7], before_k) and torch.equal(gc.rel[4, 7, 7], before_rel)
        assert torch.all(out[4, 7, 14:16] == 0) and torch.isfinite(out.float()).all()
    finally:
        ctx.set_tuning(0, 0)


def test_empty_and_full_items(ctx):
    """len == 0 without append gives zeros and -inf; a full item refuses the append, is left untouched and
    reports LETHE_ERR_CAPACITY."""
    from paper_2511_06029_b200 import binding
    L, B, Hq, Hkv, D, cap = 1, 2, 8, 2, 128, 32
    lens = torch.tensor([[[0, 5], [32, 31]]])
    oc = random_cache(L, B, Hq, Hkv, D, cap, lens, dtype=torch.bfloat16, seed=3, rel_init="rand")
    gc = to_device(oc)
    g = torch.Generator().manual_seed(1)
    q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
    scale = torch.tensor([0.1])
    _step(ctx, oc, gc, q, None, None, None, scale, 0.9, 0, 1)           # empty item: out 0, lse -inf
    before = gc.k.clone(), gc.rel.clone(), gc.len.clone()
    kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16).cuda()
    out = torch.full((L, B, Hq, D), 7.0, dtype=torch.bfloat16, device="cuda")
    ctx.decode_attend(gc, 0, 1, q.cuda(), kn, kn, torch.tensor([9, 9], dtype=torch.int32).cuda(), [0.1], 0.9, out)
    st, item = ctx.poll_status()
    assert st == binding.ERR_CAPACITY and item == 2                    # (l0, b1, h0) is the full one
    assert torch.equal(gc.len.cpu(), torch.tensor([[[1, 6], [32, 32]]], dtype=torch.int32))
    assert torch.equal(gc.k[0, 1, 0], before[0][0, 1, 0]) and torch.equal(gc.rel[0, 1, 0], before[1][0, 1, 0])
    assert torch.all(out[0, 1, :4] == 0)
    assert ctx.poll_status()[0] == 0                                     # the status word was cleared


@pytest.mark.parametrize("variant", [1, 2, 9, 18, 26, 32, 44])
def test_paged_decode_and_prune_parity(ctx, variant):
    """16-token pages behind a shuffled page table: decode steps and prune rounds, call by call."""
    w = synth.shrink(synth.WORKLOADS["ragged"], n_layers=2, batch=3, prompt_len=200)
    cap = 256
    st_c = synth.initial_kv(w, 200, cap)
    st_c["len"][0, 0, 0] = 33; st_c["len"][1, 1, 1] = 16; st_c["len"][1, 0, 0] = 1; st_c["len"][0, 2, 3] = 177
    st_p = synth.to_paged(st_c, 16, seed=3, spare_pages=7)
    oc = cache_from_state(w, st_p, cap)
    gc = to_device(oc)
    scale = synth.layer_scales(w)
    T = torch.tensor([150 * 2, 90 * 2, 400 * 2], dtype=torch.int64)
    ctx.set_tuning(variant, 2 if (variant < 8 or variant >= 44) else (3 if variant >= 32 else 0))
    try:
        for step in range(6):
            x = synth.step_inputs(w, step)
            _step(ctx, oc, gc, x["q"], x["k_new"], x["v_new"], x["token_pos"], scale, 0.95, 0, 2)
            if step in (2, 5):
                _prune_both(ctx, oc, gc, T, 12, 8, 4, cap)
    finally:
        ctx.set_tuning(0, 0)


def _prune_both(ctx, oc, gc, T, k_min, recent, sink, max_k):
    """One prune round on both sides from identical state; integer results must be bit-exact."""
    dev = gc.device
    sync_state(gc, oc)                                   # selection runs on the oracle's fp32 scores
    S_g = torch.zeros((oc.n_layers, oc.batch), dtype=torch.float32, device=dev)
    ctx.estimate_sparsity(gc, S_g)
    st, S_o = oracle.estimate_sparsity(oc)
    assert torch.allclose(S_g.cpu(), S_o, rtol=1e-3, atol=1e-6)
    bud_g = torch.zeros((oc.n_layers, oc.batch), dtype=torch.int32, device=dev)
    ctx.alloc_budgets(S_o.to(dev), T.to(dev), k_min, bud_g)          # budgets bit-exact given the oracle's S
    st, bud_o = oracle.alloc_budgets(S_o, T, k_min)
    assert st == oracle.OK and torch.equal(bud_g.cpu(), bud_o)
    keep_g = torch.full((oc.n_layers, oc.batch, oc.n_kv_heads, max_k), -7, dtype=torch.int32, device=dev)
    ctx.rasr_prune(gc, bud_g, recent, sink, keep_g)
    st_o, keep_o = oracle.rasr_prune(oc, bud_o, recent, sink, max_k=max_k)
    st_g, _ = ctx.poll_status()
    assert st_g == (3 if st_o == oracle.ERR_BUDGET else 0)
    assert torch.equal(keep_g.cpu(), keep_o)                           # retained index sets bit-exact
    assert_state_matches(gc, oc, exact_rel=True)
    return bud_o, keep_o


@pytest.mark.parametrize("dtype,D", [(torch.float32, 64), (torch.bfloat16, 128), (torch.bfloat16, 64), (torch.float32, 128)])
def test_prune_round_parity(ctx, dtype, D):
    """Sparsity within tolerance; budgets, keep_idx, len and moved rows bit-exact, with ties, items that are not
    pruned, items whose protected set exceeds the budget, and lengths around the block size."""
    L, B, Hq, Hkv, cap = 4, 3, 8, 2, 1500
    lens = _lens(L, B, Hkv, cap, seed=D, special=(1, 2, 511, 512, 513, 1024, 1499, 40, 7))
    oc = random_cache(L, B, Hq, Hkv, D, cap, lens, dtype=dtype, seed=5, rel_init="rand")
    oc.rel[oc.rel > 0.8] = 0.5                                         # many ties at the top
    oc.rel[0, 0, 0] = 0.0                                              # an all-equal item
    gc = to_device(oc)
    T = torch.tensor([4 * 300, 4 * 40, 4 * 1400], dtype=torch.int64)
    _prune_both(ctx, oc, gc, T, 36, 32, 4, cap)
    # second round on the survivors (multi-round pruning), tighter
    T2 = torch.tensor([4 * 100, 4 * 38, 4 * 600], dtype=torch.int64)
    _prune_both(ctx, oc, gc, T2, 36, 32, 4, cap)


def test_budget_edge_cases(ctx):
    from paper_2511_06029_b200 import binding
    dev = torch.device("cuda")
    for case in [([0.0, 0.5, 0.5, 0.75], 103, 2), ([0.25, 0.25, 0.25], 17, 5), ([float("nan"), 1.0, 2.0, -1.0], 1000, 0)]:
        S = torch.tensor(case[0], dtype=torch.float32)[:, None]
        T = torch.tensor([case[1]], dtype=torch.int64)
        out = torch.zeros((len(case[0]), 1), dtype=torch.int32, device=dev)
        ctx.alloc_budgets(S.to(dev), T.to(dev), case[2], out)
        st, ref = oracle.alloc_budgets(S, T, case[2])
        assert st == oracle.OK and torch.equal(out.cpu(), ref) and int(out.sum()) == case[1]
    g = torch.Generator().manual_seed(3)
    S = torch.rand((64, 5), generator=g); T = torch.randint(64 * 70, 64 * 3000, (5,), generator=g, dtype=torch.int64)
    out = torch.zeros((64, 5), dtype=torch.int32, device=dev)
    ctx.alloc_budgets(S.to(dev), T.to(dev), 68, out)
    assert torch.equal(out.cpu(), oracle.alloc_budgets(S, T, 68)[1])
    # total below the floor: every layer gets k_min and the status word says so
    ctx.alloc_budgets(S.to(dev), torch.full((5,), 10, dtype=torch.int64, device=dev), 68, out)
    st, _ = ctx.poll_status()
    assert st == binding.ERR_BUDGET and torch.all(out == 68)


def test_invalid_arguments_touch_nothing(ctx):
    from paper_2511_06029_b200 import binding
    oc = random_cache(1, 1, 8, 2, 128, 32, 8, dtype=torch.bfloat16, seed=0)
    gc = to_device(oc)
    q = torch.zeros((1, 1, 8, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.full_like(q, 3.0)
    for kwargs in [dict(gamma=0.0), dict(gamma=1.5), dict(l1=2), dict(scale=[float("nan")])]:
        with pytest.raises(binding.LetheError) as e:
            ctx.decode_attend(gc, 0, kwargs.get("l1", 1), q, None, None, None, kwargs.get("scale", [0.1]),
                              kwargs.get("gamma", 0.9), out)
        assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.LetheError):
        ctx.decode_attend(gc, 0, 1, q, q, None, None, [0.1], 0.9, out)       # k_new without v_new
    assert torch.all(out == 3.0) and torch.equal(gc.len.cpu(), oc.len)
    assert ctx.poll_status()[0] == 0


def test_tiny_workload_trajectory(ctx):
    """The Tiny configuration end to end: every call compared from identical state (call-by-call), and a
    free-running GPU trajectory whose retained sets are compared with the oracle's at the end."""
    w = synth.WORKLOADS["tiny"]
    cap = w.prompt_len + w.prune_interval
    scale = synth.layer_scales(w)
    T = torch.tensor([w.total_budget], dtype=torch.int64)
    oc = cache_from_state(w, synth.initial_kv(w, w.prompt_len, cap), cap)
    gc = to_device(oc)
    free = to_device(oc)
    dev = gc.device
    for step in range(w.gen_steps):
        x = synth.step_inputs(w, step)
        _step(ctx, oc, gc, x["q"], x["k_new"], x["v_new"], x["token_pos"], scale, w.gamma, 0, 1)
        out = torch.empty_like(x["q"], device=dev)
        ctx.decode_attend(free, 0, 1, x["q"].to(dev), x["k_new"].to(dev), x["v_new"].to(dev), x["token_pos"].to(dev),
                          scale.tolist(), w.gamma, out)
        if (step + 1) % w.prune_interval == 0:
            _prune_both(ctx, oc, gc, T, w.k_min, w.recent, w.sink, cap)
            S = torch.zeros((1, 1), dtype=torch.float32, device=dev); bud = torch.zeros((1, 1), dtype=torch.int32, device=dev)
            ctx.estimate_sparsity(free, S); ctx.alloc_budgets(S, T.to(dev), w.k_min, bud)
            ctx.rasr_prune(free, bud, w.recent, w.sink)
    assert ctx.poll_status()[0] == 0
    assert torch.equal(free.len.cpu(), oc.len)
    for h in range(w.n_kv_heads):
        a = set(free.pos[0, 0, h, :int(oc.len[0, 0, h])].cpu().tolist()); b = set(oc.pos[0, 0, h, :int(oc.len[0, 0, h])].tolist())
        jac = len(a & b) / len(a | b)
        print(f"tiny free-running retained-set Jaccard, head {h}: {jac:.4f}")
        assert jac > 0.95


@pytest.mark.parametrize("name,batch,steps", [("llama8b", 2, 10), ("qwen7b", 2, 6)])
def test_model_shaped_workloads_call_by_call(ctx, name, batch, steps):
    """Model-shaped geometry (all layers, full head counts, bf16) on a sub-batch of sequences, warm-started at
    the mean budget; decode steps with the default tuning plus two prune rounds."""
    w = synth.shrink(synth.WORKLOADS[name], batch=batch, prune_interval=steps // 2)
    n0 = 300
    cap = n0 + steps + 16
    oc = cache_from_state(w, synth.initial_kv(w, n0, cap), cap)
    gc = to_device(oc)
    scale = synth.layer_scales(w)
    T = torch.full((batch,), w.n_layers * 200, dtype=torch.int64)
    for step in range(steps):
        x = synth.step_inputs(w, step)
        _step(ctx, oc, gc, x["q"], x["k_new"], x["v_new"], x["token_pos"], scale, w.gamma, 0, w.n_layers, want_lse=False)
        if (step + 1) % w.prune_interval == 0:
            bud, _ = _prune_both(ctx, oc, gc, T, w.k_min, w.recent, w.sink, cap)
            assert int(bud.sum()) == int(T.sum())


def test_long_reasoning_shape_call_by_call(ctx):
    """Long-reasoning geometry (Llama shape, budget 2048 per layer): one sequence, all 32 layers, items above
    2000 tokens, default tuning; decode steps and a prune round."""
    oracle.set_threads(min(8, oracle.max_threads()))
    try:
        w = synth.shrink(synth.WORKLOADS["longreason"], batch=1, prune_interval=3)
        n0, cap = 2100, 2128
        oc = cache_from_state(w, synth.initial_kv(w, n0, cap), cap)
        gc = to_device(oc)
        scale = synth.layer_scales(w)
        T = torch.full((1,), w.n_layers * 2048, dtype=torch.int64)
        for step in range(4):
            x = synth.step_inputs(w, step)
            _step(ctx, oc, gc, x["q"], x["k_new"], x["v_new"], x["token_pos"], scale, w.gamma, 0, w.n_layers, want_lse=False)
            if step == 2:
                _prune_both(ctx, oc, gc, T, w.k_min, w.recent, w.sink, cap)
    finally:
        oracle.set_threads(1)


def test_ragged_paged_long_items(ctx):
    """Ragged-batch geometry (Qwen shape, 16-token pages, shuffled page tables) with the shortest and the longest
    sequence of the workload (1024 and 32768 tokens): decode steps, then a prune to a quarter of the length,
    then decode steps on the pruned cache.  Long items take the clustered kernel (16 CTAs per item)."""
    oracle.set_threads(min(8, oracle.max_threads()))
    try:
        w = synth.shrink(synth.WORKLOADS["ragged"], n_layers=2, batch=3, prompt_len=32768)
        lens = torch.tensor([1024, 32768, 9001])
        cap = 33280                                    # 2080 pages per item
        st_c = synth.initial_kv(w, 32768, cap)
        st_c["len"][:] = lens[None, :, None].to(torch.int32)
        st_p = synth.to_paged(st_c, 16, seed=5, spare_pages=11)
        del st_c
        oc = cache_from_state(w, st_p, cap)
        gc = to_device(oc)
        scale = synth.layer_scales(w)
        T = (w.n_layers * (lens // 4)).to(torch.int64)
        for step in range(4):
            x = synth.step_inputs(w, step)
            _step(ctx, oc, gc, x["q"], x["k_new"], x["v_new"], x["token_pos"], scale, w.gamma, 0, w.n_layers, want_lse=False)
            if step == 1:
                _prune_both(ctx, oc, gc, T, w.k_min, w.recent, w.sink, 9000)
    finally:
        oracle.set_threads(1)


def test_ragged_paged_many_items_default_kernel(ctx):
    """Ragged-batch geometry with enough items for the default choice to be the persistent kernel (320 items, G = 7,
    16-token pages with shuffled tables, lengths from 400 to 6000 tokens): most items are longer than the on-chip
    logit buffer, so the tail's logits go through scratch.  Decode steps, a prune to a third of each sequence's
    length, decode steps on the pruned cache."""
    oracle.set_threads(min(16, oracle.max_threads()))
    try:
        w = synth.shrink(synth.WORKLOADS["ragged"], n_layers=4, batch=20, prompt_len=6000)
        cap = 6016
        g = torch.Generator().manual_seed(77)
        lens = torch.randint(400, 6001, (20,), generator=g)
        lens[:4] = torch.tensor([400, 6000, 2047, 2049])
        st_c = synth.initial_kv(w, 6000, cap)
        st_c["len"][:] = lens[None, :, None].to(torch.int32)
        st_p = synth.to_paged(st_c, 16, seed=6, spare_pages=9)
        del st_c
        oc = cache_from_state(w, st_p, cap)
        gc = to_device(oc)
        scale = synth.layer_scales(w)
        T = (w.n_layers * (lens // 3)).to(torch.int64)
        for step in range(3):
            x = synth.step_inputs(w, step)
            _step(ctx, oc, gc, x["q"], x["k_new"], x["v_new"], x["token_pos"], scale, w.gamma, 0, w.n_layers, want_lse=False)
            if step == 0:
                _prune_both(ctx, oc, gc, T, w.k_min, w.recent, w.sink, 2048)
    finally:
        oracle.set_threads(1)


@pytest.mark.parametrize("variant,Hq,Hkv,cap", [(9, 28, 4, 3000), (12, 16, 4, 4200), (14, 28, 4, 6000), (16, 28, 4, 3000),
                                                (18, 16, 4, 4200), (20, 28, 4, 6000), (26, 16, 4, 4200)])
def test_persistent_logit_overflow(ctx, variant, Hq, Hkv, cap):
    """Items longer than the on-chip logit buffer of the persistent kernel: the logits of the tail tokens
    overflow to global scratch and the relevance update must still be exact."""
    oracle.set_threads(min(8, oracle.max_threads()))
    try:
        L, B, D = 2, 4, 128
        lens = _lens(L, B, Hkv, cap - 4, seed=cap, special=(cap - 5, cap - 300, 17, 1800, 2048, 1))
        oc = random_cache(L, B, Hq, Hkv, D, cap, lens, dtype=torch.bfloat16, seed=variant, rel_init="rand")
        gc = to_device(oc)
        ctx.set_tuning(variant, 0)
        g = torch.Generator().manual_seed(8)
        scale = torch.tensor([0.09, 0.05], dtype=torch.float32)
        for step in range(3):
            q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
            kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
            vn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
            _step(ctx, oc, gc, q, kn, vn, torch.arange(B, dtype=torch.int32) + 10 * step, scale, 0.9, 0, L)
    finally:
        ctx.set_tuning(0, 0)
        oracle.set_threads(1)


def test_free_running_overlap_llama_shape(ctx):
    """End to end on its own scores: the GPU runs a Llama-8B-shaped trajectory (2 sequences, all layers, three
    prune rounds) without being re-synchronised to the oracle; the retained sets of both are compared at the
    end.  Budgets and lengths must agree exactly whenever the fp32 sparsities round to the same weights; the
    retained sets may differ only where two scores are within the bf16/fp32 rounding of each other."""
    oracle.set_threads(min(8, oracle.max_threads()))
    try:
        w = synth.shrink(synth.WORKLOADS["llama8b"], batch=2, prune_interval=8)
        n0, cap = 260, 300
        oc = cache_from_state(w, synth.initial_kv(w, n0, cap), cap)
        gc = to_device(oc)
        dev = gc.device
        scale = synth.layer_scales(w)
        T = torch.full((2,), w.n_layers * 180, dtype=torch.int64)
        S = torch.zeros((w.n_layers, 2), dtype=torch.float32, device=dev)
        bud = torch.zeros((w.n_layers, 2), dtype=torch.int32, device=dev)
        for step in range(24):
            x = synth.step_inputs(w, step)
            st, *_ = oracle.decode_attend(oc, 0, w.n_layers, x["q"], x["k_new"], x["v_new"], x["token_pos"], scale, w.gamma)
            assert st == oracle.OK
            out = torch.empty_like(x["q"], device=dev)
            ctx.decode_attend(gc, 0, w.n_layers, x["q"].to(dev), x["k_new"].to(dev), x["v_new"].to(dev),
                              x["token_pos"].to(dev), scale.tolist(), w.gamma, out)
            if (step + 1) % w.prune_interval == 0:
                oracle_prune_round(oc, T, w.k_min, w.recent, w.sink)
                ctx.estimate_sparsity(gc, S); ctx.alloc_budgets(S, T.to(dev), w.k_min, bud)
                ctx.rasr_prune(gc, bud, w.recent, w.sink)
        assert ctx.poll_status()[0] == 0
        glen, olen = gc.len.cpu(), oc.len
        same_len = (glen == olen).float().mean().item()
        jac = []
        gpos, opos = gc.pos.cpu(), oc.pos
        for l in range(w.n_layers):
            for b in range(2):
                for h in range(w.n_kv_heads):
                    a = set(gpos[l, b, h, :int(glen[l, b, h])].tolist()); o = set(opos[l, b, h, :int(olen[l, b, h])].tolist())
                    jac.append(len(a & o) / max(1, len(a | o)))
        jac = torch.tensor(jac)
        print(f"free-running llama8b-shaped: items with equal length {same_len:.3f}; retained-set Jaccard "
              f"min {jac.min():.4f} mean {jac.mean():.4f}")
        assert jac.mean() > 0.97 and jac.min() > 0.8
    finally:
        oracle.set_threads(1)


@pytest.mark.parametrize("pinned", [True, False])
@pytest.mark.parametrize("L,B,Hkv", [(2, 2, 2), (5, 16, 20)])
def test_host_entry_point_against_the_oracle(ctx, L, B, Hkv, pinned):
    """lethe_decode_attend_host (host tensors in, host tensors out) against the oracle at the same tolerances as the
    device entry point.  Page-locked buffers: the kernel writes the results into them itself, and the large call
    (persistent kernel) also reads its inputs from them; pageable buffers: staged copies, the small call on one
    stream, the large one as two chunks whose copies overlap the kernels.  One step delivers its results into the
    middle of a larger page-locked allocation, one into a page-locked buffer that is not 16-byte aligned (which
    must take the staged path instead of being refused)."""
    pin = (lambda t: t.pin_memory()) if pinned else (lambda t: t)
    G, D, cap, n0 = 4, 64, 96, 70
    Hq = Hkv * G
    oc = random_cache(L, B, Hq, Hkv, D, cap, n0, dtype=torch.bfloat16, seed=L + B, rel_init="rand")
    gb = to_device(oc)
    g = torch.Generator().manual_seed(11)
    scale = torch.full((L,), 0.12)
    for step in range(4):
        q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
        kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
        vn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
        tp = torch.arange(B, dtype=torch.int32) + 100 + step
        s, o_out, o_lse, _ = oracle.decode_attend(oc, 0, L, q, kn, vn, tp, scale, 0.9, want_lse=True)
        assert s == oracle.OK
        qh, kh, vh, th = pin(q), pin(kn), pin(vn), pin(tp)
        if pinned and step == 1:   # results into the middle of a larger page-locked allocation
            big = torch.empty((3 * q.numel(),), dtype=torch.bfloat16).pin_memory()
            out_b = big[q.numel():2 * q.numel()].view(q.shape)
        elif pinned and step == 2:  # page-locked but only 2-byte aligned: staged, not refused
            big = torch.empty((q.numel() + 8,), dtype=torch.bfloat16).pin_memory()
            out_b = big[1:1 + q.numel()].view(q.shape)
            assert out_b.data_ptr() % 16 != 0
        else:
            out_b = pin(torch.empty_like(q))
        lse_b = pin(torch.empty((L, B, Hq), dtype=torch.float32))
        ctx.decode_attend_host(gb, 0, L, qh, kh, vh, th, scale.tolist(), 0.9, out_b, lse_b)
        assert ctx.poll_status()[0] == 0                       # synchronises the stream: host results are valid
        assert (out_b.double() - o_out.double()).abs().max() <= OUT_TOL[torch.bfloat16]
        assert torch.allclose(lse_b, o_lse, rtol=1e-4, atol=1e-4)
        assert_state_matches(gb, oc)                           # appended rows, pos, len bit-exact; rel within 1e-3 rel
    # attend-only through the host path
    q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
    s, o_out, _, _ = oracle.decode_attend(oc, 0, L, q, None, None, None, scale, 0.9)
    out_b = pin(torch.empty_like(q))
    ctx.decode_attend_host(gb, 0, L, pin(q), None, None, None, scale.tolist(), 0.9, out_b, None)
    assert ctx.poll_status()[0] == 0
    assert (out_b.double() - o_out.double()).abs().max() <= OUT_TOL[torch.bfloat16]
    assert_state_matches(gb, oc)


def test_host_entry_point_checks_before_it_enqueues(ctx):
    """Host-detectable errors of lethe_decode_attend_host are found before anything is staged or copied: the
    cache, the results and the status word stay as they were."""
    from paper_2511_06029_b200 import binding
    oc = random_cache(4, 2, 8, 2, 128, 32, 8, dtype=torch.bfloat16, seed=0)
    gc = to_device(oc)
    q = torch.zeros((4, 2, 8, 128), dtype=torch.bfloat16)
    kn = torch.zeros((4, 2, 2, 128), dtype=torch.bfloat16)
    tp = torch.zeros(2, dtype=torch.int32)
    out = torch.full_like(q, 3.0)
    for kwargs in [dict(gamma=0.0), dict(gamma=1.5), dict(scale=[0.1, float("nan"), 0.1, 0.1]), dict(l1=5)]:
        with pytest.raises(binding.LetheError) as e:
            ctx.decode_attend_host(gc, 0, kwargs.get("l1", 4), q, kn, kn, tp, kwargs.get("scale", [0.1] * 4),
                                   kwargs.get("gamma", 0.9), out)
        assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.LetheError):
        ctx.decode_attend_host(gc, 0, 4, q, kn, None, tp, [0.1] * 4, 0.9, out)      # k_new without v_new
    torch.cuda.synchronize()
    assert torch.all(out == 3.0) and torch.equal(gc.len.cpu(), oc.len) and torch.equal(gc.k.cpu().view(torch.int16), oc.k.view(torch.int16))
    assert ctx.poll_status()[0] == 0


@pytest.mark.parametrize("ratio", [0.05, 0.1, 0.25, 0.5])
def test_ragged_sweep_ratios_shortest_and_longest(ctx, ratio):
    """The ragged workload's budget ratios: the shortest and the longest sequence (1024 and 32768 tokens, 16-token
    pages, shuffled tables) attend at full length, are pruned to `ratio` of their length (never below the protected
    count: at 0.05 the short sequence's budget is the floor), and attend again on the pruned cache — every call
    against the oracle."""
    oracle.set_threads(min(8, oracle.max_threads()))
    try:
        w = synth.shrink(synth.WORKLOADS["ragged"], n_layers=2, batch=2, prompt_len=32768)
        lens = torch.tensor([1024, 32768])
        cap = 33280
        st_c = synth.initial_kv(w, 32768, cap)
        st_c["len"][:] = lens[None, :, None].to(torch.int32)
        st_p = synth.to_paged(st_c, 16, seed=int(ratio * 100), spare_pages=11)
        del st_c
        oc = cache_from_state(w, st_p, cap)
        gc = to_device(oc)
        scale = synth.layer_scales(w)
        T = (w.n_layers * torch.clamp((lens.double() * ratio).long(), min=w.k_min)).to(torch.int64)
        for step in range(4):
            x = synth.step_inputs(w, step)
            _step(ctx, oc, gc, x["q"], x["k_new"], x["v_new"], x["token_pos"], scale, w.gamma, 0, w.n_layers, want_lse=False)
            if step == 1:
                bud, _ = _prune_both(ctx, oc, gc, T, w.k_min, w.recent, w.sink, int(32770 * ratio) + 8)
                assert int(bud.sum()) == int(T.sum())
                assert torch.all(oc.len[:, 1].sum(0) == int(T[1]))      # every head of the long sequence holds its budgets
    finally:
        oracle.set_threads(1)


@pytest.mark.parametrize("variant,splits", [(0, 0), (44, 4), (45, 2), (47, 1)])
def test_layer_by_layer_launches_with_pipelining(ctx, variant, splits):
    """The way a model issues the step: one launch per layer, with the layer pipelining on (a launch fetches cached
    K / V tiles before the previous layer's launch has completed).  Several steps and a prune round in between; a
    second context-free check: the same layer twice in a row must not take the early fetch (its own previous
    launch appended to the same items), which the results would show as a stale length."""
    w = synth.shrink(synth.WORKLOADS["llama8b"], n_layers=6, batch=3, prune_interval=4)
    n0, cap = 333, 352
    oc = cache_from_state(w, synth.initial_kv(w, n0, cap), cap)
    oc.len[2, 1, 3] = 15; oc.len[4, 0, 0] = 1; oc.len[5, 2, 7] = 348
    gc = to_device(oc)
    dev = gc.device
    scale = synth.layer_scales(w)
    T = torch.full((3,), w.n_layers * 200, dtype=torch.int64)
    ctx.set_tuning(variant, splits)
    ctx.set_tuning(51, 0)
    try:
        for step in range(8):
            x = synth.step_inputs(w, step)
            s, o_out, _, _ = oracle.decode_attend(oc, 0, w.n_layers, x["q"], x["k_new"], x["v_new"], x["token_pos"], scale, w.gamma)
            assert s == oracle.OK
            out = torch.full_like(x["q"], float("nan"), device=dev)
            q, kn, vn, tp = (x[k].to(dev) for k in ("q", "k_new", "v_new", "token_pos"))
            for l in range(w.n_layers):                              # back to back, nothing in between
                ctx.decode_attend(gc, l, l + 1, q[l:l + 1], kn[l:l + 1], vn[l:l + 1], tp, scale.tolist(), w.gamma, out[l:l + 1])
            assert ctx.poll_status()[0] == 0
            assert (out.cpu().double() - o_out.double()).abs().max() <= OUT_TOL[torch.bfloat16]
            assert_state_matches(gc, oc)
            if (step + 1) % w.prune_interval == 0:
                _prune_both(ctx, oc, gc, T, w.k_min, w.recent, w.sink, cap)
        # the same layer twice in a row: the second launch depends on the first one's append
        for rep in range(2):
            x = synth.step_inputs(w, 100 + rep)
            s, o_out, _, _ = oracle.decode_attend(oc, 3, 4, x["q"][3:4], x["k_new"][3:4], x["v_new"][3:4], x["token_pos"], scale, w.gamma)
            out = torch.zeros_like(x["q"][3:4], device=dev)
            ctx.decode_attend(gc, 3, 4, x["q"][3:4].to(dev), x["k_new"][3:4].to(dev), x["v_new"][3:4].to(dev),
                              x["token_pos"].to(dev), scale.tolist(), w.gamma, out)
        assert ctx.poll_status()[0] == 0
        assert (out.cpu().double() - o_out.double()).abs().max() <= OUT_TOL[torch.bfloat16]
        assert_state_matches(gc, oc)
    finally:
        ctx.set_tuning(50, 0)
        ctx.set_tuning(0, 0)
