"""GPU parity of lethe_prefill_seed (relevance of the prompt from the causal prefill attention, Eq. 2 with Q > 1
folded through Eq. 5) against the oracle: |d| <= 1e-3 |ref| + 1e-6 on rel[0..P), everything else untouched."""
import pytest
import torch

import oracle
from helpers import cache_from_state, gpu_context, random_cache, to_device
from paper_2511_06029_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = gpu_context()
    yield c
    c.close()


TCGEN05, MMA_SYNC, TCGEN05_CP_ASYNC = 40, 41, 42                     # lethe_set_tuning codes of the engines


@pytest.mark.parametrize("engine", [TCGEN05, MMA_SYNC, TCGEN05_CP_ASYNC])
@pytest.mark.parametrize("Hq,Hkv,D,P", [(32, 8, 128, 300), (28, 4, 128, 129), (8, 8, 128, 64), (4, 2, 64, 257),
                                        (6, 2, 128, 17), (5, 1, 64, 1), (16, 2, 128, 200), (8, 2, 128, 128),
                                        (14, 2, 64, 385), (10, 2, 128, 200), (12, 2, 64, 150)])
def test_prefill_seed_parity(ctx, engine, Hq, Hkv, D, P):
    oracle.set_threads(min(8, oracle.max_threads()))
    ctx.set_tuning(engine, 0)
    try:
        L, B, cap = 2, 2, max(320, P + 16)
        lens = torch.full((L, B, Hkv), P, dtype=torch.int32)
        lens[0, 0, 0] = min(cap, P + 7)                               # a longer item: slots beyond P stay as they are
        oc = random_cache(L, B, Hq, Hkv, D, cap, lens, dtype=torch.bfloat16, seed=P, rel_init="rand")
        gc = to_device(oc)
        g = torch.Generator().manual_seed(P + Hq)
        qp = torch.randn((L, B, P, Hq, D), generator=g).to(torch.bfloat16)
        scale = torch.tensor([0.09, 0.2], dtype=torch.float32) * (128 / D) ** 0.5
        before = oc.clone()
        assert oracle.prefill_seed(oc, qp, scale, 0.97) == oracle.OK
        ctx.prefill_seed(gc, qp.cuda(), scale.tolist(), 0.97)
        assert ctx.poll_status()[0] == 0
        got = gc.rel.cpu()
        assert torch.allclose(got[..., :P], oc.rel[..., :P], rtol=1e-3, atol=1e-6), \
            f"max abs diff {(got[..., :P] - oc.rel[..., :P]).abs().max().item()}"
        assert torch.equal(got[..., P:], before.rel[..., P:])
        assert torch.equal(gc.k.cpu().view(torch.int16), before.k.view(torch.int16)) and torch.equal(gc.len.cpu(), before.len)
        # total mass of every item: G (1 - gamma^P) / (1 - gamma)
        G = Hq // Hkv
        want = G * (1 - 0.97 ** P) / (1 - 0.97)
        assert torch.allclose(got[..., :P].double().sum(-1), torch.full((L, B, Hkv), want, dtype=torch.float64), rtol=2e-3)
    finally:
        oracle.set_threads(1)
        ctx.set_tuning(TCGEN05, 0)


@pytest.mark.parametrize("engine", [TCGEN05, MMA_SYNC])
def test_prefill_seed_paged_then_decode(ctx, engine):
    """Paged cache: seed the prompt's relevance, then continue with decode steps; both sides stay in step."""
    oracle.set_threads(min(8, oracle.max_threads()))
    ctx.set_tuning(engine, 0)
    try:
        w = synth.shrink(synth.WORKLOADS["ragged"], n_layers=2, batch=2, prompt_len=150)
        cap = 192
        st_p = synth.to_paged(synth.initial_kv(w, 150, cap), 16, seed=4, spare_pages=5)
        oc = cache_from_state(w, st_p, cap)
        gc = to_device(oc)
        dev = gc.device
        g = torch.Generator().manual_seed(77)
        qp = torch.randn((w.n_layers, 2, 150, w.n_q_heads, w.head_dim), generator=g).to(torch.bfloat16)
        scale = synth.layer_scales(w)
        assert oracle.prefill_seed(oc, qp, scale, w.gamma) == oracle.OK
        ctx.prefill_seed(gc, qp.to(dev), scale.tolist(), w.gamma)
        assert torch.allclose(gc.rel.cpu()[..., :150], oc.rel[..., :150], rtol=1e-3, atol=1e-6)
        gc.rel.copy_(oc.rel)
        for step in range(3):
            x = synth.step_inputs(w, step)
            st, ref, _, _ = oracle.decode_attend(oc, 0, w.n_layers, x["q"], x["k_new"], x["v_new"], x["token_pos"], scale, w.gamma)
            out = torch.empty_like(x["q"], device=dev)
            ctx.decode_attend(gc, 0, w.n_layers, x["q"].to(dev), x["k_new"].to(dev), x["v_new"].to(dev),
                              x["token_pos"].to(dev), scale.tolist(), w.gamma, out)
            assert (out.cpu().float() - ref.float()).abs().max() <= 2e-2
            assert torch.allclose(gc.rel.cpu(), oc.rel, rtol=1e-3, atol=1e-6)
        assert ctx.poll_status()[0] == 0
    finally:
        oracle.set_threads(1)
        ctx.set_tuning(TCGEN05, 0)


def test_prefill_seed_engines_agree_on_a_long_prompt(ctx):
    """Prompt of several tiles per operand (P = 1100, G = 7 padded to 8 columns per query): the two engines run the
    same arithmetic in a different summation order."""
    L, B, Hq, Hkv, D, P, cap = 1, 2, 14, 2, 128, 1100, 1120
    oc = random_cache(L, B, Hq, Hkv, D, cap, P, dtype=torch.bfloat16, seed=5, rel_init="rand")
    qp = torch.randn((L, B, P, Hq, D), generator=torch.Generator().manual_seed(6)).to(torch.bfloat16).cuda()
    res = {}
    for engine in (TCGEN05, MMA_SYNC, TCGEN05_CP_ASYNC):
        gc = to_device(oc)
        ctx.set_tuning(engine, 0)
        ctx.prefill_seed(gc, qp, [0.11], 0.995)
        assert ctx.poll_status()[0] == 0
        res[engine] = gc.rel.cpu()
    ctx.set_tuning(TCGEN05, 0)
    assert torch.allclose(res[TCGEN05][..., :P], res[MMA_SYNC][..., :P], rtol=2e-4, atol=1e-7)
    assert torch.allclose(res[TCGEN05_CP_ASYNC][..., :P], res[MMA_SYNC][..., :P], rtol=2e-4, atol=1e-7)
    assert torch.equal(res[TCGEN05][..., P:], oc.rel[..., P:])
    G = Hq // Hkv
    want = G * (1 - 0.995 ** P) / (1 - 0.995)
    assert torch.allclose(res[TCGEN05][..., :P].double().sum(-1), torch.full((L, B, Hkv), want, dtype=torch.float64), rtol=2e-3)


@pytest.mark.parametrize("engine", [TCGEN05, MMA_SYNC, TCGEN05_CP_ASYNC])
def test_prefill_seed_capacity_below_one_tile(ctx, engine):
    """A cache whose capacity is smaller than the 128-row operand tile (the tile runs past the item's rows)."""
    L, B, Hq, Hkv, D, P, cap = 2, 3, 8, 2, 128, 40, 48
    oc = random_cache(L, B, Hq, Hkv, D, cap, 44, dtype=torch.bfloat16, seed=12, rel_init="rand")
    gc = to_device(oc)
    qp = torch.randn((L, B, P, Hq, D), generator=torch.Generator().manual_seed(13)).to(torch.bfloat16)
    scale = torch.tensor([0.09, 0.12], dtype=torch.float32)
    before = oc.clone()
    assert oracle.prefill_seed(oc, qp, scale, 0.95) == oracle.OK
    ctx.set_tuning(engine, 0)
    try:
        ctx.prefill_seed(gc, qp.cuda(), scale.tolist(), 0.95)
        assert ctx.poll_status()[0] == 0
    finally:
        ctx.set_tuning(TCGEN05, 0)
    got = gc.rel.cpu()
    assert torch.allclose(got[..., :P], oc.rel[..., :P], rtol=1e-3, atol=1e-6)
    assert torch.equal(got[..., P:], before.rel[..., P:])


def test_prefill_seed_rejects_bad_input(ctx):
    from paper_2511_06029_b200 import binding
    oc = random_cache(1, 1, 4, 1, 64, 64, 20, dtype=torch.bfloat16, seed=0, rel_init="rand")
    gc = to_device(oc)
    qp = torch.zeros((1, 1, 30, 4, 64), dtype=torch.bfloat16, device="cuda")
    ctx.prefill_seed(gc, qp, [0.1], 0.9)                                 # len 20 < P 30: skipped and reported
    st, item = ctx.poll_status()
    assert st == binding.ERR_CAPACITY and item == 0
    assert torch.equal(gc.rel.cpu(), oc.rel)
    with pytest.raises(binding.LetheError):
        ctx.prefill_seed(gc, qp, [0.1], 1.5)
    oc32 = random_cache(1, 1, 4, 1, 64, 64, 40, dtype=torch.float32, seed=0)
    with pytest.raises(binding.LetheError) as e:
        ctx.prefill_seed(to_device(oc32), qp.float(), [0.1], 0.9)
    assert e.value.status == binding.ERR_UNSUPPORTED
