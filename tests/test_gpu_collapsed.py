"""GPU parity of lethe_collapsed_prune (retention by the head- and batch-collapsed score of Eq. 2) against the
oracle: the shared retention set, every item's moved rows and the lengths are integer / bit-exact results; the
fp32 sum that decides them is taken in the same order on both sides."""
import pytest
import torch

import oracle
from helpers import assert_state_matches, cache_from_state, gpu_context, random_cache, sync_state, to_device
from paper_2511_06029_b200 import binding, synth

pytestmark = pytest.mark.gpu

HEADS, BATCH = oracle.COLLAPSE_HEADS, oracle.COLLAPSE_HEADS_BATCH


@pytest.fixture(scope="module")
def ctx():
    c = gpu_context()
    yield c
    c.close()


def _both(ctx, oc, gc, budgets, recent, sink, scope, max_k, expect=oracle.OK):
    groups = budgets.numel()
    keep_g = torch.full((groups, max_k), -7, dtype=torch.int32, device=gc.device)
    ctx.collapsed_prune(gc, budgets.to(gc.device), recent, sink, scope, keep_g)
    st_o, keep_o = oracle.collapsed_prune(oc, budgets, recent, sink, scope, max_k=max_k)
    assert st_o == expect and ctx.poll_status()[0] == expect
    assert torch.equal(keep_g.cpu(), keep_o), "retained slots differ"
    assert_state_matches(gc, oc, exact_rel=True)
    return keep_o


def test_constants_agree():
    assert (binding.COLLAPSE_HEADS, binding.COLLAPSE_HEADS_BATCH) == (HEADS, BATCH)


@pytest.mark.parametrize("scope", [HEADS, BATCH])
@pytest.mark.parametrize("dtype,D,Hkv", [(torch.bfloat16, 128, 8), (torch.float32, 64, 3), (torch.bfloat16, 64, 1)])
def test_collapsed_prune_parity(ctx, scope, dtype, D, Hkv):
    """Groups of equal length around the block size (one length per group), heavy-tailed scores with ties and
    exact zeros, budgets below / inside / above the length, two rounds in a row."""
    L, B, cap = 4, 3, 1500
    g = torch.Generator().manual_seed(100 * scope + D + Hkv)
    if scope == HEADS:
        per = torch.randint(1, cap, (L, B, 1), generator=g)
        per.view(-1)[:7] = torch.tensor([1, 2, 511, 512, 513, 1025, 1499])
        lens = per.expand(L, B, Hkv).contiguous()
        budgets = torch.randint(0, cap, (L * B,), generator=g, dtype=torch.int32)
        budgets[:4] = torch.tensor([1, 1, 37, 512], dtype=torch.int32)
    else:
        per = torch.tensor([513, 1499, 40, 1024]).reshape(L, 1, 1)
        lens = per.expand(L, B, Hkv).contiguous()
        budgets = torch.tensor([100, 700, 41, 1023], dtype=torch.int32)
    oc = random_cache(L, B, Hkv * 2, Hkv, D, cap, lens, dtype=dtype, seed=Hkv + scope, rel_init="rand")
    oc.rel.pow_(6).mul_(3.0)
    oc.rel[oc.rel < 1e-5] = 0.0
    oc.rel[1] = (oc.rel[1] * 8).round() / 8                          # coarse values: many equal sums
    oc.pos += torch.arange(B, dtype=torch.int32).reshape(1, B, 1, 1) * 1000   # rows differ between sequences
    gc = to_device(oc)
    expect = oracle.OK
    keep = _both(ctx, oc, gc, budgets, 0, 0, scope, cap)
    assert (keep >= 0).sum() > 0
    # second round on the survivors with protected slots (budgets may now fall below them: same flag on both sides)
    budgets2 = torch.clamp(budgets // 2, min=40)
    _both(ctx, oc, gc, budgets2, 32, 4, scope, cap, expect)


def test_collapsed_prune_flags(ctx):
    oc = random_cache(2, 2, 4, 2, 64, 128, 100, dtype=torch.bfloat16, seed=2, rel_init="rand")
    # a group whose heads are out of step is refused and untouched; the others are pruned
    oc.len[1, 0, 1] = 99
    gc = to_device(oc)
    _both(ctx, oc, gc, torch.tensor([30, 30, 30, 30], dtype=torch.int32), 8, 2, HEADS, 128, oracle.ERR_INVALID_ARG)
    assert oc.len[1, 0].tolist() == [100, 99]
    # protected set above the budget
    oc = random_cache(2, 2, 4, 2, 64, 128, 100, dtype=torch.bfloat16, seed=3, rel_init="rand")
    gc = to_device(oc)
    _both(ctx, oc, gc, torch.tensor([5, 60], dtype=torch.int32), 8, 2, BATCH, 128, oracle.ERR_BUDGET)
    assert oc.len[0].flatten().tolist() == [10] * 4
    # host-side argument checks enqueue nothing
    with pytest.raises(binding.LetheError):
        ctx.collapsed_prune(gc, torch.zeros(2, dtype=torch.int32, device=gc.device), 8, 2, 2)
    with pytest.raises(binding.LetheError):
        ctx.collapsed_prune(gc, torch.zeros(2, dtype=torch.int32, device=gc.device), -1, 2, BATCH)


def test_collapsed_prune_fp32_sum_order(ctx):
    """The case in which the fp32 head-by-head sum and the exact sum pick different slots."""
    big = float(2 ** 24)
    oc = random_cache(1, 1, 3, 3, 64, 8, 5, dtype=torch.bfloat16, seed=1)
    oc.rel[0, 0, :, :5] = torch.tensor([[0, big, big, 0, 0], [0, 1, 2, 0, 0], [0, 1, 0, 0, 0]])
    gc = to_device(oc)
    keep = _both(ctx, oc, gc, torch.tensor([3], dtype=torch.int32), 1, 1, HEADS, 8)
    assert [i for i in keep[0].tolist() if i >= 0] == [0, 2, 4]


def test_collapsed_prune_long_group_keys_in_global_scratch(ctx):
    """A group longer than the shared-memory key buffer (keys and list in global scratch)."""
    n, cap = 70000, 70016
    oc = random_cache(1, 1, 2, 2, 64, cap, n, dtype=torch.bfloat16, seed=6, rel_init="rand")
    oc.rel[0, 0, :, 1000:30000] = 0.125
    gc = to_device(oc)
    _both(ctx, oc, gc, torch.tensor([20000], dtype=torch.int32), 64, 4, HEADS, 20000)


def test_collapsed_prune_paged_in_the_decode_loop(ctx):
    """Decode steps accumulate relevance in a paged cache (Qwen-7B-shaped geometry), every few steps the sequences
    are pruned with the collapsed score; call-by-call parity."""
    w = synth.shrink(synth.WORKLOADS["ragged"], n_layers=2, batch=2, prompt_len=150)
    cap = 256
    st_p = synth.to_paged(synth.initial_kv(w, 150, cap), 16, seed=5, spare_pages=3)
    st_p["len"][:] = 150                                             # one length per sequence
    oc = cache_from_state(w, st_p, cap)
    gc = to_device(oc)
    dev = gc.device
    scale = synth.layer_scales(w)
    for step in range(12):
        x = synth.step_inputs(w, step)
        st, ref, _, _ = oracle.decode_attend(oc, 0, w.n_layers, x["q"], x["k_new"], x["v_new"], x["token_pos"], scale, 0.95)
        assert st == oracle.OK
        out = torch.empty_like(x["q"], device=dev)
        ctx.decode_attend(gc, 0, w.n_layers, x["q"].to(dev), x["k_new"].to(dev), x["v_new"].to(dev),
                          x["token_pos"].to(dev), scale.tolist(), 0.95, out)
        assert (out.cpu().float() - ref.float()).abs().max() <= 2e-2
        assert_state_matches(gc, oc)
        if step % 4 == 3:
            sync_state(gc, oc)                                        # selection on the oracle's fp32 scores
            budgets = torch.tensor([90, 120, 70, 170], dtype=torch.int32)
            _both(ctx, oc, gc, budgets, 16, 4, HEADS, cap)
    assert int(oc.len.min()) < 150 and int(oc.len.max()) == 150 + 12   # three groups pruned, one never over budget
