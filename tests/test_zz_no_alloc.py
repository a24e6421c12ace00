"""lethe_rasr_prune_static — the prune step for callers that are not allowed to allocate device memory (for
example a server whose memory pool owns the whole GPU, so that no lethe_ctx can be created) — must give exactly
what lethe_rasr_prune gives.  Called through the C ABI, twice in a row, because every call reuses the same
in-library scratch and finds the previous call's contents there.  Collected last on purpose."""
import pytest
import torch

from helpers import gpu_context, random_cache, to_device

pytestmark = pytest.mark.gpu


def _state(seed, dtype, D):
    L, B, Hq, Hkv, cap = 3, 2, 8, 2, 1500
    g = torch.Generator().manual_seed(seed)
    lens = torch.randint(1, cap, (L, B, Hkv), generator=g)
    lens.view(-1)[:6] = torch.tensor([1, 511, 512, 513, 1499, 40])
    oc = random_cache(L, B, Hq, Hkv, D, cap, lens, dtype=dtype, seed=seed, rel_init="rand")
    oc.rel[oc.rel > 0.8] = 0.5          # ties at the top
    oc.rel[0, 0, 0] = 0.0               # an all-equal item
    return oc


@pytest.mark.parametrize("dtype,D", [(torch.bfloat16, 128), (torch.float32, 64)])
def test_static_prune_matches_context_prune_twice(dtype, D):
    from paper_2511_06029_b200 import binding
    ctx = gpu_context()
    try:
        oc = _state(11, dtype, D)
        ref, new = to_device(oc), to_device(oc)
        dev = ref.device
        L, B, Hkv, cap = oc.n_layers, oc.batch, oc.n_kv_heads, oc.capacity
        rounds = [torch.tensor([[300, 40], [1400, 36], [700, 5]], dtype=torch.int32),      # 5 < sink + recent
                  torch.tensor([[100, 38], [600, 36], [90, 36]], dtype=torch.int32)]
        for rnd, budgets in enumerate(rounds):
            bud = budgets.to(dev)
            keep_ref = torch.full((L, B, Hkv, cap), -7, dtype=torch.int32, device=dev)
            keep_new = torch.full((L, B, Hkv, cap), -9, dtype=torch.int32, device=dev)
            ctx.rasr_prune(ref, bud, 32, 4, keep_ref)
            st_ref, item_ref = ctx.poll_status()
            status = torch.full((2,), 77, dtype=torch.int32, device=dev)
            rc = binding.rasr_prune_static(new, bud, 32, 4, keep_new, status)
            assert rc == binding.OK
            torch.cuda.synchronize()
            # the status code must agree; which of several offending items reports first is a race on both sides
            assert status.tolist()[0] == st_ref, (rnd, status.tolist(), st_ref, item_ref)
            if rnd == 0:
                assert st_ref == binding.ERR_BUDGET and status.tolist()[1] in (10, 11)   # items of (layer 2, sequence 1)
            assert torch.equal(keep_new, keep_ref), f"round {rnd}: kept slots differ"
            assert torch.equal(new.len, ref.len)
            for l in range(L):
                for b in range(B):
                    for h in range(Hkv):
                        n = int(ref.len[l, b, h])
                        for name in ("k", "v", "rel", "pos"):
                            a = getattr(new, name)[l, b, h, :n]; r = getattr(ref, name)[l, b, h, :n]
                            assert torch.equal(a.view(torch.uint8), r.view(torch.uint8)), (rnd, name, l, b, h)
    finally:
        ctx.close()


def test_static_prune_rejects_what_its_scratch_cannot_hold():
    from paper_2511_06029_b200 import binding
    gpu_context().close()
    dev = torch.device("cuda", 0)
    L, B, Hkv, D = 2, 2, 2, 64
    cap = binding.STATIC_PRUNE_MAX_ENTRIES // (L * B * Hkv) + 1          # one slot too many
    k = torch.zeros((L, B, Hkv, cap, D), dtype=torch.bfloat16, device=dev)
    rel = torch.rand((L, B, Hkv, cap), device=dev)
    pos = torch.zeros((L, B, Hkv, cap), dtype=torch.int32, device=dev)
    ln = torch.full((L, B, Hkv), 100, dtype=torch.int32, device=dev)
    cache = binding.Cache(4, k, k.clone(), rel, pos, ln)
    bud = torch.full((L, B), 10, dtype=torch.int32, device=dev)
    assert binding.rasr_prune_static(cache, bud, 2, 1) == binding.ERR_TOO_LARGE
    torch.cuda.synchronize()
    assert torch.all(ln == 100)                                           # nothing ran
    fit = binding.Cache(4, k[..., :cap - 1, :].contiguous(), k[..., :cap - 1, :].contiguous(),
                        rel[..., :cap - 1].contiguous(), pos[..., :cap - 1].contiguous(), ln)
    assert binding.rasr_prune_static(fit, bud, 2, 1) == binding.OK        # exactly at the limit is accepted
    torch.cuda.synchronize()
    assert torch.all(ln == 10)
