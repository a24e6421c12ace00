"""GPU parity of the quantised-cache path (K / V as e4m3 bytes with per-layer scales, bf16 activations) against the
oracle: appended rows are quantised to the same bytes, outputs within 2e-2, relevance within 1e-3 relative, and the
prune round moves the bytes exactly as the oracle does."""
import pytest
import torch

import oracle
from helpers import assert_state_matches, gpu_context, oracle_prune_round, sync_state, to_device
from paper_2511_06029_b200 import binding, synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = gpu_context()
    yield c
    c.close()


FMT = {"e4m3": (torch.float8_e4m3fn, 448.0), "e5m2": (torch.float8_e5m2, 57344.0)}


def fp8_cache(L, B, Hq, Hkv, D, cap, lens, seed, k_scale=None, v_scale=None, page_tokens=0, fmt="e4m3"):
    """Quantised cache drawn as the quantisation of Gaussian K / V (a few keys enlarged, as the workloads' anchors)."""
    f8, fmax = FMT[fmt]
    g = torch.Generator().manual_seed(seed)
    ks = torch.tensor(k_scale if k_scale is not None else [1.0] * L, dtype=torch.float32)
    vs = torch.tensor(v_scale if v_scale is not None else [1.0] * L, dtype=torch.float32)
    k = torch.randn((L, B, Hkv, cap, D), generator=g)
    k[:, :, :, ::17] *= 3.0
    v = torch.randn((L, B, Hkv, cap, D), generator=g)
    k8 = (k / ks.reshape(L, 1, 1, 1, 1)).clamp(-fmax, fmax).to(f8)
    v8 = (v / vs.reshape(L, 1, 1, 1, 1)).clamp(-fmax, fmax).to(f8)
    rel = torch.rand((L, B, Hkv, cap), generator=g)
    pos = torch.arange(cap, dtype=torch.int32).expand(L, B, Hkv, cap).contiguous()
    ln = torch.full((L, B, Hkv), lens, dtype=torch.int32) if isinstance(lens, int) else lens.to(torch.int32).contiguous()
    if page_tokens:
        assert cap % page_tokens == 0
        pages_per_item = cap // page_tokens
        n_pages = L * B * Hkv * pages_per_item + 3
        perm = torch.randperm(n_pages, generator=g)[:L * B * Hkv * pages_per_item].to(torch.int32)
        table = perm.reshape(L, B, Hkv, pages_per_item).contiguous()
        pool_k = torch.zeros((n_pages, page_tokens, D), dtype=torch.uint8)
        pool_v = torch.zeros((n_pages, page_tokens, D), dtype=torch.uint8)
        pool_k[table.long().flatten()] = k8.view(torch.uint8).reshape(-1, page_tokens, D)
        pool_v[table.long().flatten()] = v8.view(torch.uint8).reshape(-1, page_tokens, D)
        return oracle.OracleCache(L, B, Hq, Hkv, D, pages_per_item, pool_k.view(f8), pool_v.view(f8),
                                  rel, pos, ln, page_tokens, table, k_scale=ks, v_scale=vs)
    return oracle.OracleCache(L, B, Hq, Hkv, D, cap, k8, v8, rel, pos, ln, k_scale=ks, v_scale=vs)


def _step(ctx, oc, gc, q, kn, vn, tp, scale, gamma, want_lse=False):
    L = oc.n_layers
    st, ref, lse_ref, _ = oracle.decode_attend(oc, 0, L, q, kn, vn, tp, scale, gamma, want_lse=want_lse)
    dev = gc.device
    out = torch.empty_like(q, device=dev)
    lse = torch.empty((L, oc.batch, oc.n_q_heads), dtype=torch.float32, device=dev) if want_lse else None
    ctx.decode_attend(gc, 0, L, q.to(dev), None if kn is None else kn.to(dev), None if vn is None else vn.to(dev),
                      None if tp is None else tp.to(dev), scale.tolist(), gamma, out, lse)
    assert st == oracle.OK and ctx.poll_status()[0] == 0
    # 2e-2 absolute for outputs of the usual size; outputs made large by a saturated value row (up to 448 * scale)
    # carry the bf16 rounding of their own magnitude (2^-8 relative)
    d = (out.cpu().float() - ref.float()).abs()
    assert bool((d <= 2e-2 + 2.0 ** -7 * ref.float().abs()).all()), f"attention output error {d.max().item()}"
    if want_lse:
        assert torch.allclose(lse.cpu(), lse_ref, rtol=1e-4, atol=1e-4)
    assert_state_matches(gc, oc)           # appended bytes, pos, len bit-exact; rel within 1e-3


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
@pytest.mark.parametrize("paged", [False, True])
@pytest.mark.parametrize("Hq,Hkv,D", [(8, 2, 128), (7, 1, 128), (4, 4, 64), (16, 2, 64), (6, 2, 128)])
def test_quantised_decode_parity(ctx, Hq, Hkv, D, paged, fmt):
    """Ragged lengths over several 16-token groups and tails, attend-only and appending steps, scales that are not
    powers of two, a new token beyond the representable range (saturates)."""
    L, B, cap = 2, 3, 208
    g = torch.Generator().manual_seed(Hq * 10 + D)
    lens = torch.randint(1, cap - 8, (L, B, Hkv), generator=g)
    lens.view(-1)[:4] = torch.tensor([1, 15, 16, 17])[: min(4, lens.numel())]
    oc = fp8_cache(L, B, Hq, Hkv, D, cap, lens, seed=Hq + D, k_scale=[0.37, 1.5], v_scale=[2.25, 0.6],
                   page_tokens=16 if paged else 0, fmt=fmt)
    gc = to_device(oc)
    scale = torch.tensor([0.11, 0.07], dtype=torch.float32) * (128 / D) ** 0.5
    for step in range(5):
        q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
        if step == 1:
            _step(ctx, oc, gc, q, None, None, None, scale, 0.95, want_lse=True)
            continue
        kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
        vn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
        if step == 2:
            big = 1e4 if fmt == "e4m3" else 1e6                      # beyond the format's range: saturates
            kn[0, 0, 0, :3] = torch.tensor([big, -big, 165.5], dtype=torch.bfloat16)
            vn[1, 1, 0, :2] = torch.tensor([-0.3 * big, 269.0], dtype=torch.bfloat16)
        _step(ctx, oc, gc, q, kn, vn, torch.arange(B, dtype=torch.int32) + 300 + step, scale, 0.95)


@pytest.mark.parametrize("variant,splits,fmt", [(2, 1, "e4m3"), (3, 2, "e4m3"), (4, 4, "e4m3"), (5, 1, "e4m3"), (6, 8, "e4m3"),
                                                (7, 2, "e4m3"), (0, 0, "e4m3"), (8, 0, "e4m3"), (9, 0, "e4m3"), (10, 1, "e4m3"),
                                                (11, 0, "e4m3"), (12, 0, "e4m3"), (13, 0, "e4m3"),
                                                (2, 1, "e5m2"), (3, 2, "e5m2"), (4, 4, "e5m2"), (5, 1, "e5m2"), (6, 8, "e5m2"),
                                                (7, 2, "e5m2"), (0, 0, "e5m2"), (9, 0, "e5m2")])
def test_quantised_decode_shapes_and_clusters(ctx, variant, splits, fmt):
    """Every kernel shape and cluster size on items long enough to give every CTA of a cluster several groups."""
    L, B, Hq, Hkv, D, cap = 1, 2, 8, 2, 128, 1100
    g = torch.Generator().manual_seed(variant * 7 + splits)
    lens = torch.tensor([[[1037, 700], [513, 1090]]])
    oc = fp8_cache(L, B, Hq, Hkv, D, cap, lens, seed=variant, k_scale=[0.8], v_scale=[1.25], fmt=fmt)
    gc = to_device(oc)
    ctx.set_tuning(variant, splits)
    try:
        scale = torch.tensor([0.09], dtype=torch.float32)
        for step in range(2):
            q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
            kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
            vn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
            _step(ctx, oc, gc, q, kn, vn, torch.tensor([5, 6], dtype=torch.int32), scale, 0.99)
    finally:
        ctx.set_tuning(0, 0)


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
def test_quantised_trajectory_with_prune_rounds(ctx, fmt):
    """Llama-8B-shaped geometry (2 layers, 2 sequences): decode steps with appends, a prune round every 6 steps on
    the oracle's scores; bytes, positions and lengths stay identical throughout."""
    oracle.set_threads(min(8, oracle.max_threads()))
    try:
        w = synth.shrink(synth.WORKLOADS["llama8b"], n_layers=2, batch=2)
        L, B, Hq, Hkv, D, cap, n0 = 2, 2, w.n_q_heads, w.n_kv_heads, w.head_dim, 320, 270
        oc = fp8_cache(L, B, Hq, Hkv, D, cap, n0, seed=21, k_scale=[0.5, 0.7], v_scale=[0.9, 1.1], fmt=fmt)
        oc.rel.zero_()
        gc = to_device(oc)
        dev = gc.device
        scale = synth.layer_scales(w)
        T = torch.full((B,), L * 200, dtype=torch.int64)
        S = torch.zeros((L, B), dtype=torch.float32, device=dev)
        bud = torch.zeros((L, B), dtype=torch.int32, device=dev)
        keep = torch.zeros((L, B, Hkv, cap), dtype=torch.int32, device=dev)
        for step in range(18):
            x = synth.step_inputs(w, step)
            _step(ctx, oc, gc, x["q"], x["k_new"], x["v_new"], x["token_pos"], scale, w.gamma)
            if step % 6 == 5:
                sync_state(gc, oc)                                   # selection on the oracle's fp32 scores
                st, S_o, bud_o, keep_o = oracle_prune_round(oc, T, w.k_min, w.recent, w.sink, max_k=cap)
                assert st == oracle.OK
                ctx.estimate_sparsity(gc, S); ctx.alloc_budgets(S, T.to(dev), w.k_min, bud)
                ctx.rasr_prune(gc, bud, w.recent, w.sink, keep)
                assert ctx.poll_status()[0] == 0
                assert torch.equal(bud.cpu(), bud_o) and torch.equal(keep.cpu(), keep_o)
                assert_state_matches(gc, oc, exact_rel=True)
        assert int(oc.len.sum()) <= B * Hkv * (L * 200 + L * 6)          # every sequence was cut back to its total budget
    finally:
        oracle.set_threads(1)


def test_quantised_cache_limits(ctx):
    oc = fp8_cache(1, 1, 4, 1, 64, 32, 32, seed=1)
    gc = to_device(oc)
    q = torch.zeros((1, 1, 4, 64), dtype=torch.bfloat16, device="cuda")
    kn = torch.zeros((1, 1, 1, 64), dtype=torch.bfloat16, device="cuda")
    out = torch.empty_like(q)
    ctx.decode_attend(gc, 0, 1, q, kn, kn, torch.zeros(1, dtype=torch.int32, device="cuda"), [0.1], 0.9, out)
    st, item = ctx.poll_status()
    assert st == binding.ERR_CAPACITY and item == 0 and int(gc.len[0, 0, 0]) == 32        # full: untouched, reported
    with pytest.raises(binding.LetheError) as e:                                          # prompt seeding: bf16 caches only
        ctx.prefill_seed(gc, torch.zeros((1, 1, 8, 4, 64), dtype=torch.bfloat16, device="cuda"), [0.1], 0.9)
    assert e.value.status == binding.ERR_UNSUPPORTED
    bad = binding.Cache(4, gc.k, gc.v, gc.rel, gc.pos, gc.len, k_scale=[0.0], v_scale=[1.0])
    with pytest.raises(binding.LetheError) as e:
        ctx.decode_attend(bad, 0, 1, q, None, None, None, [0.1], 0.9, out)
    assert e.value.status == binding.ERR_INVALID_ARG


@pytest.mark.parametrize("paged", [False, True])
def test_quantised_persistent_kernel_many_items(ctx, paged):
    """The persistent kernel (forced: shape (12,3)) on more than two items per SM, then the automatic choice on the
    same state: ragged lengths, appends, an attend-only step."""
    L, B, Hq, Hkv, D, cap = 4, 10, 16, 8, 128, 160
    g = torch.Generator().manual_seed(31 + paged)
    lens = torch.randint(1, cap - 6, (L, B, Hkv), generator=g)
    oc = fp8_cache(L, B, Hq, Hkv, D, cap, lens, seed=5, k_scale=[0.4, 0.6, 0.8, 1.0], v_scale=[1.0, 0.5, 2.0, 0.75],
                   page_tokens=16 if paged else 0)
    gc = to_device(oc)
    scale = torch.tensor([0.1, 0.08, 0.12, 0.09], dtype=torch.float32)
    try:
        for step in range(5):
            ctx.set_tuning(9 if step < 3 else 0, 0)
            q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
            if step == 2:
                _step(ctx, oc, gc, q, None, None, None, scale, 0.97, want_lse=True)
                continue
            kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
            vn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
            _step(ctx, oc, gc, q, kn, vn, torch.arange(B, dtype=torch.int32) + 500 + step, scale, 0.97)
    finally:
        ctx.set_tuning(0, 0)


def test_quantised_persistent_kernel_logit_overflow(ctx):
    """Items longer than the on-chip logit buffer of the widest shape: the tail's logits go through global scratch."""
    L, B, Hq, Hkv, D, cap = 1, 2, 16, 2, 128, 12000
    g = torch.Generator().manual_seed(3)
    lens = torch.tensor([[[11950, 9000], [4000, 11990]]])
    oc = fp8_cache(L, B, Hq, Hkv, D, cap, lens, seed=9, k_scale=[0.5], v_scale=[1.5])
    gc = to_device(oc)
    ctx.set_tuning(12, 0)                                     # (16 warps, 2 stages): least room for logits
    try:
        for step in range(2):
            q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
            kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
            vn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
            _step(ctx, oc, gc, q, kn, vn, torch.tensor([1, 2], dtype=torch.int32), torch.tensor([0.05]), 0.99)
    finally:
        ctx.set_tuning(0, 0)


@pytest.mark.parametrize("pinned", [True, False])
def test_quantised_host_entry_point(ctx, pinned):
    """lethe_decode_attend_host on a quantised cache against the oracle: page-locked buffers (the kernel reads its
    inputs from them and writes the results into them) and pageable ones (staged copies)."""
    L, B, Hq, Hkv, D, cap = 2, 3, 8, 2, 128, 112
    g = torch.Generator().manual_seed(5)
    lens = torch.randint(1, cap - 8, (L, B, Hkv), generator=g)
    oc = fp8_cache(L, B, Hq, Hkv, D, cap, lens, seed=9, k_scale=[0.37, 1.5], v_scale=[2.25, 0.6], fmt="e4m3")
    gc = to_device(oc)
    pin = (lambda t: t.pin_memory()) if pinned else (lambda t: t)
    scale = torch.tensor([0.11, 0.07], dtype=torch.float32)
    for step in range(3):
        q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
        kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
        vn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
        tp = torch.arange(B, dtype=torch.int32) + 50 + step
        st, ref, lse_ref, _ = oracle.decode_attend(oc, 0, L, q, kn, vn, tp, scale, 0.95, want_lse=True)
        out = pin(torch.empty_like(q))
        lse = pin(torch.empty((L, B, Hq), dtype=torch.float32))
        ctx.decode_attend_host(gc, 0, L, pin(q), pin(kn), pin(vn), pin(tp), scale.tolist(), 0.95, out, lse)
        assert st == oracle.OK and ctx.poll_status()[0] == 0      # the poll synchronises the stream
        d = (out.float() - ref.float()).abs()
        assert bool((d <= 2e-2 + 2.0 ** -7 * ref.float().abs()).all()), f"attention output error {d.max().item()}"
        assert torch.allclose(lse, lse_ref, rtol=1e-4, atol=1e-4)
        assert_state_matches(gc, oc)


TENSOR_MEMORY = 14                                                   # lethe_set_tuning code of the tcgen05 kernel


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
@pytest.mark.parametrize("paged", [False, True])
@pytest.mark.parametrize("Hq,Hkv", [(8, 2), (7, 1), (16, 2), (5, 5), (24, 4), (10, 2)])
def test_quantised_tensor_memory_kernel(ctx, Hq, Hkv, paged, fmt):
    """The tcgen05 kernel (cache bytes straight into the MMAs, queries and probabilities as three e4m3 terms) on
    G = 4, 7, 8, 1, 6, 5: lengths around the 128-token tile (1, 127, 128, 129, 255, 256, 257), several tiles per item,
    appending and attend-only steps, a new token beyond the representable range, an empty and a full item."""
    L, B, D, cap = 2, 3, 128, 416
    g = torch.Generator().manual_seed(Hq * 10 + paged)
    lens = torch.randint(1, cap - 8, (L, B, Hkv), generator=g)
    special = torch.tensor([1, 127, 128, 129, 255, 256, 257, 400])
    lens.view(-1)[:min(8, lens.numel())] = special[:min(8, lens.numel())]
    oc = fp8_cache(L, B, Hq, Hkv, D, cap, lens, seed=Hq + 3, k_scale=[0.37, 1.5], v_scale=[2.25, 0.6],
                   page_tokens=16 if paged else 0, fmt=fmt)
    gc = to_device(oc)
    scale = torch.tensor([0.11, 0.07], dtype=torch.float32)
    ctx.set_tuning(TENSOR_MEMORY, 0)
    try:
        for step in range(5):
            q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
            if step == 1:
                _step(ctx, oc, gc, q, None, None, None, scale, 0.95, want_lse=True)
                continue
            kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
            vn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
            if step == 2:
                big = 1e4 if fmt == "e4m3" else 1e6
                kn[0, 0, 0, :3] = torch.tensor([big, -big, 165.5], dtype=torch.bfloat16)
                vn[1, 1, 0, :2] = torch.tensor([-0.3 * big, 269.0], dtype=torch.bfloat16)
            _step(ctx, oc, gc, q, kn, vn, torch.arange(B, dtype=torch.int32) + 300 + step, scale, 0.95, want_lse=(step == 3))
        # an empty item (attend only) and a full one (append refused) in the same launches
        oc.len[0, 1, 0] = 0; oc.len[1, 2, Hkv - 1] = cap
        sync_state(gc, oc)
        q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
        _step(ctx, oc, gc, q, None, None, None, scale, 0.95, want_lse=True)
        kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16).cuda()
        out = torch.full((L, B, Hq, D), 7.0, dtype=torch.bfloat16, device="cuda")
        before = gc.k.clone()
        ctx.decode_attend(gc, 0, L, q.cuda(), kn, kn, torch.zeros(B, dtype=torch.int32).cuda(), scale.tolist(), 0.95, out)
        st, item = ctx.poll_status()
        assert st == binding.ERR_CAPACITY and item == (1 * B + 2) * Hkv + Hkv - 1
        assert int(gc.len[1, 2, Hkv - 1]) == cap and int(gc.len[0, 1, 0]) == 1
        G = Hq // Hkv
        assert torch.all(out[1, 2, (Hkv - 1) * G:] == 0) and torch.isfinite(out.float()).all()
        if not paged:
            assert torch.equal(gc.k[1, 2, Hkv - 1].view(torch.uint8), before[1, 2, Hkv - 1].view(torch.uint8))
    finally:
        ctx.set_tuning(0, 0)


@pytest.mark.parametrize("paged", [False, True])
def test_quantised_tensor_memory_kernel_many_and_long_items(ctx, paged):
    """More items than SMs (every CTA walks several through its queue and the ring runs across item boundaries),
    with a few items of twenty tiles among short ones; uninitialised-looking bytes (NaN patterns) beyond the items'
    ends must not leak into the results."""
    L, B, Hq, Hkv, D, cap = 3, 9, 16, 8, 128, 2624
    g = torch.Generator().manual_seed(17 + paged)
    lens = torch.randint(1, 300, (L, B, Hkv), generator=g)
    n_long = len(lens.view(-1)[::37])
    lens.view(-1)[::37] = torch.randint(2000, cap - 8, (n_long,), generator=g)
    oc = fp8_cache(L, B, Hq, Hkv, D, cap, lens, seed=5, k_scale=[0.4, 0.6, 0.8], v_scale=[1.0, 0.5, 2.0],
                   page_tokens=16 if paged else 0)
    if not paged:                                                    # poison the rows beyond every item's end
        idx = torch.arange(cap)[None, None, None, :] > lens[..., None] + 2
        oc.k.view(torch.uint8)[idx] = 0x7F
        oc.v.view(torch.uint8)[idx] = 0xFF
    gc = to_device(oc)
    scale = torch.tensor([0.1, 0.08, 0.12], dtype=torch.float32)
    ctx.set_tuning(TENSOR_MEMORY, 0)
    try:
        for step in range(3):
            q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
            if step == 1:
                _step(ctx, oc, gc, q, None, None, None, scale, 0.97, want_lse=True)
                continue
            kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
            vn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
            _step(ctx, oc, gc, q, kn, vn, torch.arange(B, dtype=torch.int32) + 500 + step, scale, 0.97)
    finally:
        ctx.set_tuning(0, 0)


@pytest.mark.parametrize("paged", [False, True])
def test_quantised_automatic_choice_many_items(ctx, paged):
    """No tuning set: a launch with more than two items per SM takes the library's automatic choice for quantised
    caches.  Every item spans three or four tiles, so each CTA streams multi-tile items back to back; two prune
    rounds in between change the lengths (and the work-queue order) under the kernel."""
    L, B, Hq, Hkv, D, cap = 5, 8, 32, 8, 128, 512
    assert L * B * Hkv >= 2 * torch.cuda.get_device_properties(0).multi_processor_count
    g = torch.Generator().manual_seed(41 + paged)
    lens = torch.randint(290, 440, (L, B, Hkv), generator=g)
    oc = fp8_cache(L, B, Hq, Hkv, D, cap, lens, seed=11, k_scale=[0.4, 0.6, 0.8, 0.5, 1.0], v_scale=[1.0, 0.5, 2.0, 0.7, 0.9],
                   page_tokens=16 if paged else 0)
    oc.rel.zero_()
    gc = to_device(oc)
    scale = torch.tensor([0.1, 0.08, 0.12, 0.09, 0.1], dtype=torch.float32)
    ctx.set_tuning(0, 0)
    for step in range(6):
        q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
        kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
        vn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
        _step(ctx, oc, gc, q, kn, vn, torch.arange(B, dtype=torch.int32) + 700 + step, scale, 0.97, want_lse=(step == 4))
        if step in (1, 3):                                           # prune on the oracle's scores, as the parity bar prescribes
            gc.rel.copy_(oc.rel)
            budgets = torch.full((L, B), 200 + 40 * step, dtype=torch.int32)
            st_o, _ = oracle.rasr_prune(oc, budgets, 16, 4)
            ctx.rasr_prune(gc, budgets.cuda(), 16, 4)
            assert st_o == oracle.OK and ctx.poll_status()[0] == 0
            assert_state_matches(gc, oc, exact_rel=True)


@pytest.mark.parametrize("Hq,paged", [(64, False), (56, True), (48, False)])
def test_quantised_automatic_choice_large_capacity(ctx, Hq, paged):
    """No tuning set, many items, eight / seven / six query heads per KV head and a capacity whose logits do not fit
    on chip beside the tile rings: the automatic choice has to take a kernel that overflows them (the tail of the
    long items goes through scratch), with the same results.  A few items are nearly as long as the capacity."""
    L, B, Hkv, D, cap = 5, 8, 8, 128, 2560
    assert L * B * Hkv >= 2 * torch.cuda.get_device_properties(0).multi_processor_count
    g = torch.Generator().manual_seed(77)
    lens = torch.randint(1, 200, (L, B, Hkv), generator=g)
    n_long = len(lens.view(-1)[::53])
    lens.view(-1)[::53] = torch.randint(2300, cap - 8, (n_long,), generator=g)
    oc = fp8_cache(L, B, Hq, Hkv, D, cap, lens, seed=13, k_scale=[0.4, 0.6, 0.8, 0.5, 1.0], v_scale=[1.0, 0.5, 2.0, 0.7, 0.9],
                   page_tokens=16 if paged else 0)
    gc = to_device(oc)
    scale = torch.tensor([0.1, 0.08, 0.12, 0.09, 0.1], dtype=torch.float32)
    ctx.set_tuning(0, 0)
    for step in range(3):
        q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
        if step == 1:
            _step(ctx, oc, gc, q, None, None, None, scale, 0.97, want_lse=True)
            continue
        kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
        vn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
        _step(ctx, oc, gc, q, kn, vn, torch.arange(B, dtype=torch.int32) + 900 + step, scale, 0.97)


@pytest.mark.parametrize("variant", [TENSOR_MEMORY, 0])
def test_quantised_query_magnitudes(ctx, variant):
    """Query rows far outside e4m3's range (the tensor-memory kernel feeds the queries to the MMAs as 8-bit terms):
    heads whose rows are scaled by 2^12, 2^-20, 3e4 and 1e-7, with the softmax scale compensating so that the logits
    stay ordinary; a head of zeros; one huge element in an otherwise ordinary row."""
    L, B, Hq, Hkv, D, cap = 2, 3, 8, 2, 128, 416
    g = torch.Generator().manual_seed(91)
    lens = torch.randint(1, cap - 8, (L, B, Hkv), generator=g)
    oc = fp8_cache(L, B, Hq, Hkv, D, cap, lens, seed=17, k_scale=[0.37, 1.5], v_scale=[2.25, 0.6])
    gc = to_device(oc)
    ctx.set_tuning(variant, 0)
    try:
        for step, (mul, sc) in enumerate([(4096.0, 0.1 / 4096), (2.0 ** -20, 0.1 * 2.0 ** 20), (3.0e4, 0.08 / 3.0e4), (1.0e-7, 0.08e7)]):
            q = torch.randn((L, B, Hq, D), generator=g) * mul
            q[0, 0, 1] = 0.0                                         # a head of zeros: uniform attention
            q[1, 1, 2, 5] = 40.0 * mul                               # one element far above the rest of its row
            q = q.to(torch.bfloat16)
            kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
            vn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
            scale = torch.tensor([sc, sc * 0.7], dtype=torch.float32)
            _step(ctx, oc, gc, q, kn, vn, torch.arange(B, dtype=torch.int32) + 300 + step, scale, 0.95, want_lse=(step == 1))
    finally:
        ctx.set_tuning(0, 0)


@pytest.mark.parametrize("fmt,paged,splits", [("e4m3", False, 0), ("e4m3", True, 4), ("e5m2", False, 2)])
def test_quantised_layer_by_layer_with_pipelining(ctx, fmt, paged, splits):
    """One launch per layer on a quantised cache, with the layer pipelining on (a launch fetches cached K / V tiles
    before the previous layer's launch has completed), several appending steps, then the same layer twice in a row
    (the second launch depends on the first one's append and must not take the early fetch)."""
    L, B, Hq, Hkv, D, cap = 6, 3, 32, 8, 128, 352
    g = torch.Generator().manual_seed(23 + paged)
    lens = torch.randint(200, 330, (L, B, Hkv), generator=g)
    lens[2, 1, 3] = 15; lens[4, 0, 0] = 1; lens[5, 2, 7] = 340
    oc = fp8_cache(L, B, Hq, Hkv, D, cap, lens, seed=29, k_scale=[0.4, 0.6, 0.8, 0.5, 1.0, 0.7], v_scale=[1.0, 0.5, 2.0, 0.7, 0.9, 1.3],
                   page_tokens=16 if paged else 0, fmt=fmt)
    gc = to_device(oc)
    dev = gc.device
    scale = torch.tensor([0.1, 0.08, 0.12, 0.09, 0.1, 0.11], dtype=torch.float32)
    ctx.set_tuning(44 if splits else 0, splits)
    ctx.set_tuning(51, 0)
    try:
        for step in range(5):
            q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
            kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
            vn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
            tp = torch.arange(B, dtype=torch.int32) + 400 + step
            st, ref, _, _ = oracle.decode_attend(oc, 0, L, q, kn, vn, tp, scale, 0.97)
            assert st == oracle.OK
            out = torch.full_like(q, float("nan"), device=dev)
            qd, kd, vd, td = q.to(dev), kn.to(dev), vn.to(dev), tp.to(dev)
            for l in range(L):                                       # back to back, nothing in between
                ctx.decode_attend(gc, l, l + 1, qd[l:l + 1], kd[l:l + 1], vd[l:l + 1], td, scale.tolist(), 0.97, out[l:l + 1])
            assert ctx.poll_status()[0] == 0
            d = (out.cpu().float() - ref.float()).abs()
            assert bool((d <= 2e-2 + 2.0 ** -7 * ref.float().abs()).all()), f"attention output error {d.max().item()}"
            assert_state_matches(gc, oc)
        for rep in range(2):                                         # the same layer twice in a row
            q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
            kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
            tp = torch.arange(B, dtype=torch.int32) + 500 + rep
            st, ref, _, _ = oracle.decode_attend(oc, 3, 4, q[3:4], kn[3:4], kn[3:4], tp, scale, 0.97)
            out = torch.zeros_like(q[3:4], device=dev)
            ctx.decode_attend(gc, 3, 4, q[3:4].to(dev), kn[3:4].to(dev), kn[3:4].to(dev), tp.to(dev), scale.tolist(), 0.97, out)
        assert ctx.poll_status()[0] == 0
        d = (out.cpu().float() - ref.float()).abs()
        assert bool((d <= 2e-2 + 2.0 ** -7 * ref.float().abs()).all())
        assert_state_matches(gc, oc)
    finally:
        ctx.set_tuning(50, 0)
        ctx.set_tuning(0, 0)
