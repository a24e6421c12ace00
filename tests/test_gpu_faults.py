"""Device-side failure reporting, tested without faulting or hanging anything: bounded waits that are made to run
out by a host-set poll limit, and page ids outside the pool that the kernels range-check and never dereference.
In both cases the launch returns, the status word names the event, and the context stays usable."""
import pytest
import torch

import oracle
from helpers import assert_state_matches, cache_from_state, gpu_context, random_cache, to_device
from paper_2511_06029_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = gpu_context()
    yield c
    c.close()


def _decode_once(ctx, oc, gc, seed):
    g = torch.Generator().manual_seed(seed)
    L, B, Hq, Hkv, D = oc.n_layers, oc.batch, oc.n_q_heads, oc.n_kv_heads, oc.head_dim
    q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
    kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
    vn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
    tp = torch.arange(B, dtype=torch.int32) + 500
    scale = torch.full((L,), 0.09)
    out = torch.zeros_like(q, device="cuda")
    ctx.decode_attend(gc, 0, L, q.cuda(), kn.cuda(), vn.cuda(), tp.cuda(), scale.tolist(), 0.95, out)
    return q, kn, vn, tp, scale, out


@pytest.mark.parametrize("variant", [16, 19, 24])
def test_attend_wait_runs_out_and_the_context_recovers(ctx, variant):
    """The persistent kernel with the asynchronous epilogue (cp.async and TMA staging): with a poll limit of one
    the epilogue warps' first wait for the streaming warps gives up.  The launch must return with
    LETHE_ERR_TIMEOUT; the next ordinary launch on the same context (which needs the work queue re-armed) must be
    parity-green."""
    from paper_2511_06029_b200 import binding
    L, B, Hq, Hkv, D, cap = 2, 3, 16, 4, 128, 2600
    oc = random_cache(L, B, Hq, Hkv, D, cap, 2500, dtype=torch.bfloat16, seed=variant, rel_init="rand")
    broken, good = to_device(oc), to_device(oc)
    ctx.set_tuning(variant, 0)
    try:
        ctx.set_wait_limit(1)
        _decode_once(ctx, oc, broken, 3)
        st, where = ctx.poll_status()                           # returns: nothing hangs
        assert st == binding.ERR_TIMEOUT and 0 <= where < 148
        assert ctx.poll_status()[0] == 0                        # reported once, then cleared
        ctx.set_wait_limit(0)
        q, kn, vn, tp, scale, out = _decode_once(ctx, oc, good, 3)
        assert ctx.poll_status()[0] == 0
        s, ref, _, _ = oracle.decode_attend(oc, 0, L, q, kn, vn, tp, scale, 0.95)
        assert s == oracle.OK
        assert (out.cpu().float() - ref.float()).abs().max() <= 2e-2
        assert_state_matches(good, oc)
    finally:
        ctx.set_wait_limit(0)
        ctx.set_tuning(0, 0)
    with pytest.raises(binding.LetheError):
        ctx.set_wait_limit(-1)


@pytest.mark.parametrize("engine", [40, 42])
def test_prefill_wait_runs_out_and_the_context_recovers(ctx, engine):
    """The tensor-memory prompt-relevance kernels (TMA and cp.async producers): a poll limit of one makes the MMA
    warp's first wait for an operand tile give up; the CTAs wait for what they started, free their tensor memory
    and return LETHE_ERR_TIMEOUT.  The same call with the default limit is then parity-green."""
    from paper_2511_06029_b200 import binding
    L, B, Hq, Hkv, D, P, cap = 2, 2, 8, 2, 128, 300, 320
    oc = random_cache(L, B, Hq, Hkv, D, cap, P, dtype=torch.bfloat16, seed=engine, rel_init="rand")
    gc = to_device(oc)
    g = torch.Generator().manual_seed(engine)
    qp = torch.randn((L, B, P, Hq, D), generator=g).to(torch.bfloat16)
    scale = torch.tensor([0.09, 0.12])
    ctx.set_tuning(engine, 0)
    try:
        ctx.set_wait_limit(1)
        ctx.prefill_seed(gc, qp.cuda(), scale.tolist(), 0.97)
        st, item = ctx.poll_status()
        assert st == binding.ERR_TIMEOUT and 0 <= item < L * B * Hkv
        ctx.set_wait_limit(0)
        assert oracle.prefill_seed(oc, qp, scale, 0.97) == oracle.OK
        ctx.prefill_seed(gc, qp.cuda(), scale.tolist(), 0.97)
        assert ctx.poll_status()[0] == 0
        assert torch.allclose(gc.rel.cpu()[..., :P], oc.rel[..., :P], rtol=1e-3, atol=1e-6)
    finally:
        ctx.set_wait_limit(0)
        ctx.set_tuning(40, 0)


def test_quantised_tensor_memory_kernel_wait_runs_out(ctx):
    """The tcgen05 kernel for byte caches: with a poll limit of one its first hand-off gives up; the CTAs wait for
    the copies they started, free their tensor memory and return LETHE_ERR_TIMEOUT, and the same context then runs
    the same launch correctly."""
    from paper_2511_06029_b200 import binding
    from test_gpu_fp8 import fp8_cache, _step
    L, B, Hq, Hkv, D, cap = 2, 3, 16, 4, 128, 1600
    oc = fp8_cache(L, B, Hq, Hkv, D, cap, 1500, seed=4, k_scale=[0.5, 0.7], v_scale=[0.9, 1.1])
    broken, good = to_device(oc), to_device(oc)
    g = torch.Generator().manual_seed(2)
    q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
    kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
    scale = torch.tensor([0.09, 0.1])
    ctx.set_tuning(14, 0)
    try:
        ctx.set_wait_limit(1)
        out = torch.zeros_like(q, device="cuda")
        ctx.decode_attend(broken, 0, L, q.cuda(), kn.cuda(), kn.cuda(), torch.zeros(B, dtype=torch.int32).cuda(), scale.tolist(), 0.95, out)
        st, where = ctx.poll_status()
        assert st == binding.ERR_TIMEOUT and 0 <= where < 148
        ctx.set_wait_limit(0)
        _step(ctx, oc, good, q, kn, kn, torch.zeros(B, dtype=torch.int32), scale, 0.95)
    finally:
        ctx.set_wait_limit(0)
        ctx.set_tuning(0, 0)


def _paged_state(lens_special=()):
    w = synth.shrink(synth.WORKLOADS["ragged"], n_layers=2, batch=2, prompt_len=400)
    cap = 416
    st_c = synth.initial_kv(w, 400, cap)
    g = torch.Generator().manual_seed(1)
    st_c["rel"][:] = torch.rand(st_c["rel"].shape, generator=g)
    st_p = synth.to_paged(st_c, 16, seed=8, spare_pages=3)
    return w, cap, st_p


@pytest.mark.parametrize("call", ["rasr", "segment", "collapsed", "static"])
def test_prune_reports_a_page_id_outside_the_pool(ctx, call):
    """A page table whose item (layer 1, sequence 0, head 2) names a page beyond the pool, at a table slot that only
    a row slot other than thread 0's ever touches.  The id is range-checked on the device and never dereferenced:
    the rows that live on that page do not move, the call records LETHE_ERR_PAGE with the item, and every other
    item is pruned as the oracle prunes it."""
    from paper_2511_06029_b200 import binding
    w, cap, st_p = _paged_state()
    st_p["rel"][1, 0, :, 144:160] = 2.0                        # the rows on the bad page are certain survivors
    oc = cache_from_state(w, st_p, cap)
    bad_item = (1, 0, 2)
    flat = (bad_item[0] * 2 + bad_item[1]) * w.n_kv_heads + bad_item[2]
    gc = to_device(oc)
    table = gc.page_table.clone()
    table[bad_item][9] = gc.c.n_pages + 5                      # slots 144..159 of that item: source rows only
    bad = binding.Cache(w.n_q_heads, gc.k, gc.v, gc.rel, gc.pos, gc.len, table)
    dev = gc.device
    bud = torch.full((2, 2), 120, dtype=torch.int32)
    if call == "rasr":
        ctx.rasr_prune(bad, bud.to(dev), 16, 4)
        st, item = ctx.poll_status()
        oracle.rasr_prune(oc, bud, 16, 4)
    elif call == "static":
        status = torch.zeros(2, dtype=torch.int32, device=dev)
        assert binding.rasr_prune_static(bad, bud.to(dev), 16, 4, None, status) == binding.OK
        torch.cuda.synchronize()
        st, item = status.tolist()
        oracle.rasr_prune(oc, bud, 16, 4)
    elif call == "segment":
        le = torch.zeros((2, 2, w.n_kv_heads), dtype=torch.int32)
        ctx.segment_prune(bad, 4, 1.5, 16, 4, le.to(dev))
        st, item = ctx.poll_status()
        oracle.segment_prune(oc, 4, 1.5, 16, 4, le)
    else:
        ctx.collapsed_prune(bad, bud.to(dev), 16, 4, binding.COLLAPSE_HEADS)
        st, item = ctx.poll_status()
        oracle.collapsed_prune(oc, bud, 16, 4, 0)
    assert st == binding.ERR_PAGE and item == flat, (st, item, flat)
    assert torch.equal(gc.len.cpu(), oc.len)
    assert int(oc.len[bad_item]) < 400                          # the item was pruned, so rows did have to move
    # every other item is bit-exact; compare through the good table (the pools are shared)
    ok_g = binding.Cache(w.n_q_heads, gc.k, gc.v, gc.rel, gc.pos, gc.len, gc.page_table)
    from helpers import logical_rows
    g_rows = logical_rows(ok_g.k, ok_g.v, ok_g.rel, ok_g.pos, ok_g.len, ok_g.page_table, 16)
    o_rows = logical_rows(oc.k, oc.v, oc.rel, oc.pos, oc.len, oc.page_table, 16)
    for i, (gr, orow) in enumerate(zip(g_rows, o_rows)):
        if i == flat:
            assert torch.equal(gr[2], orow[2]) and torch.equal(gr[3], orow[3])     # rel and pos are not paged: they moved
            continue
        for a, b in zip(gr, orow):
            assert torch.equal(a.view(torch.uint8), b.view(torch.uint8)), f"item {i}"
