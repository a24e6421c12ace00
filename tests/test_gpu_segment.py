"""GPU parity of lethe_segment_prune (Algorithm 1 with the size trigger) against the oracle: breakpoints, retained
index sets, moved rows, lengths and updated thresholds are all integer / bit-exact results."""
import pytest
import torch

import oracle
from helpers import assert_state_matches, cache_from_state, gpu_context, random_cache, sync_state, to_device
from paper_2511_06029_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = gpu_context()
    yield c
    c.close()


def _segment_both(ctx, oc, gc, D, tau, recent, sink, le, max_k):
    dev = gc.device
    le_g = le.clone().to(dev)
    keep_g = torch.full((oc.n_layers, oc.batch, oc.n_kv_heads, max_k), -7, dtype=torch.int32, device=dev)
    ctx.segment_prune(gc, D, tau, recent, sink, le_g, keep_g)
    st_o, keep_o = oracle.segment_prune(oc, D, tau, recent, sink, le, max_k=max_k)
    assert st_o == oracle.OK and ctx.poll_status()[0] == 0
    assert torch.equal(le_g.cpu(), le), "eviction thresholds differ"
    assert torch.equal(keep_g.cpu(), keep_o), "retained slots differ"
    assert_state_matches(gc, oc, exact_rel=True)
    return keep_o


@pytest.mark.parametrize("dtype,D_head", [(torch.bfloat16, 128), (torch.float32, 64)])
@pytest.mark.parametrize("segments,tau", [(8, 400.0), (4, 3.0), (2, 1.0), (16, 20.0), (8, 1e30)])
def test_segment_prune_parity(ctx, dtype, D_head, segments, tau):
    """Heavy-tailed scores with ties, lengths around the block size, thresholds below / at / above the length,
    two rounds in a row (the second on the survivors and the updated thresholds)."""
    L, B, Hq, Hkv, cap = 3, 3, 8, 2, 1400
    g = torch.Generator().manual_seed(int(segments * 7 + tau) % 1000)
    lens = torch.randint(1, cap, (L, B, Hkv), generator=g)
    lens.view(-1)[:8] = torch.tensor([1, 2, 511, 512, 513, 1024, 1399, 40])
    oc = random_cache(L, B, Hq, Hkv, D_head, cap, lens, dtype=dtype, seed=segments, rel_init="rand")
    oc.rel.pow_(8).mul_(5.0)                                         # a few large scores, many tiny ones
    oc.rel[oc.rel < 1e-6] = 0.0                                      # exact zeros (ties at the bottom)
    oc.rel[0, 1, 0] = 0.25                                           # an all-equal item
    gc = to_device(oc)
    le = torch.randint(0, cap, (L, B, Hkv), generator=g, dtype=torch.int32)
    le.view(-1)[:4] = torch.tensor([0, 1, 511, 600], dtype=torch.int32)
    _segment_both(ctx, oc, gc, segments, tau, 32, 4, le, cap)
    le2 = (le // 2).contiguous()                                     # force a second trigger on most items
    _segment_both(ctx, oc, gc, segments, tau, 32, 4, le2, cap)


def test_segment_prune_in_the_decode_loop(ctx):
    """Threshold-triggered pruning inside a decode trajectory (Qwen-7B-shaped geometry, paged cache): decode steps
    accumulate relevance, every few steps Algorithm 1 runs with the running thresholds; call-by-call parity."""
    w = synth.shrink(synth.WORKLOADS["ragged"], n_layers=2, batch=2, prompt_len=180)
    cap = 256
    st_p = synth.to_paged(synth.initial_kv(w, 180, cap), 16, seed=9, spare_pages=3)
    oc = cache_from_state(w, st_p, cap)
    gc = to_device(oc)
    dev = gc.device
    scale = synth.layer_scales(w)
    le = torch.full((w.n_layers, 2, w.n_kv_heads), 150, dtype=torch.int32)
    for step in range(12):
        x = synth.step_inputs(w, step)
        st, ref, _, _ = oracle.decode_attend(oc, 0, w.n_layers, x["q"], x["k_new"], x["v_new"], x["token_pos"], scale, 0.95)
        out = torch.empty_like(x["q"], device=dev)
        ctx.decode_attend(gc, 0, w.n_layers, x["q"].to(dev), x["k_new"].to(dev), x["v_new"].to(dev),
                          x["token_pos"].to(dev), scale.tolist(), 0.95, out)
        assert (out.cpu().float() - ref.float()).abs().max() <= 2e-2
        assert_state_matches(gc, oc)
        if step % 4 == 3:
            sync_state(gc, oc)                                        # selection on the oracle's fp32 scores
            _segment_both(ctx, oc, gc, 8, 4.0, 16, 4, le, cap)
    assert int(oc.len.max()) < 180 + 12                               # something was pruned along the way


def test_segment_prune_invalid_arguments(ctx):
    from paper_2511_06029_b200 import binding
    oc = random_cache(1, 1, 4, 1, 64, 64, 50, dtype=torch.bfloat16, seed=0, rel_init="rand")
    gc = to_device(oc)
    le = torch.zeros((1, 1, 1), dtype=torch.int32, device="cuda")
    for kw in [dict(D=1), dict(tau=0.5), dict(tau=float("nan")), dict(recent=-1)]:
        with pytest.raises(binding.LetheError) as e:
            ctx.segment_prune(gc, kw.get("D", 8), kw.get("tau", 4.0), kw.get("recent", 4), 1, le)
        assert e.value.status == binding.ERR_INVALID_ARG
    assert int(gc.len[0, 0, 0]) == 50 and int(le[0, 0, 0]) == 0
