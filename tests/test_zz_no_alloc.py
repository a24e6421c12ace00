"""lethe_rasr_prune_static — the prune step for callers that are not allowed to allocate device memory (for
example a server whose memory pool owns the whole GPU, so that no lethe_ctx can be created) — must give exactly
what the oracle's retention step gives, and what lethe_rasr_prune gives.  Called through the C ABI, twice in a
row, because every call reuses the same in-library scratch and finds the previous call's contents there; the
second call must not change the device's free memory.  Collected last on purpose."""
import pytest
import torch

import oracle
from helpers import assert_state_matches, gpu_context, random_cache, to_device

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


def _paged_state(seed):
    from paper_2511_06029_b200 import synth
    from helpers import cache_from_state
    w = synth.shrink(synth.WORKLOADS["ragged"], n_layers=2, batch=3, prompt_len=1400)
    cap = 1504
    st = synth.initial_kv(w, 1400, cap)
    g = torch.Generator().manual_seed(seed)
    st["rel"][:] = torch.rand(st["rel"].shape, generator=g)
    st["len"][0, 1, 2] = 17; st["len"][1, 2, 0] = 1023
    return cache_from_state(w, synth.to_paged(st, 16, seed=seed, spare_pages=5), cap)


def _fp8_state(seed):
    from test_gpu_fp8 import fp8_cache
    g = torch.Generator().manual_seed(seed)
    lens = torch.randint(1, 600, (2, 2, 2), generator=g)
    return fp8_cache(2, 2, 8, 2, 128, 608, lens, seed, k_scale=[0.3, 0.7], v_scale=[1.1, 0.4], page_tokens=16)


def _free_bytes():
    free, _ = torch.cuda.mem_get_info()                      # cudaMemGetInfo: what the driver has left on the device
    return free


STATES = {
    "bf16": lambda: (_state(11, torch.bfloat16, 128), [[[300, 40], [1400, 36], [700, 5]], [[100, 38], [600, 36], [90, 36]]]),
    "f32": lambda: (_state(11, torch.float32, 64), [[[300, 40], [1400, 36], [700, 5]], [[100, 38], [600, 36], [90, 36]]]),
    "bf16-paged": lambda: (_paged_state(5), [[[500, 40, 1000], [1400, 36, 200]], [[100, 38, 300], [600, 36, 150]]]),
    "e4m3-paged": lambda: (_fp8_state(9), [[[300, 40], [100, 36]], [[60, 38], [50, 36]]]),
}


@pytest.mark.parametrize("kind", list(STATES))
def test_static_prune_matches_the_oracle_twice(kind):
    from paper_2511_06029_b200 import binding
    ctx = gpu_context()
    try:
        oc, rounds = STATES[kind]()
        ref, new = to_device(oc), to_device(oc)
        dev = ref.device
        L, B, Hkv = oc.n_layers, oc.batch, oc.n_kv_heads
        max_k = int(oc.len.max())
        for rnd, budgets in enumerate(rounds):
            budgets = torch.tensor(budgets, dtype=torch.int32)
            bud = budgets.to(dev)
            keep_ref = torch.full((L, B, Hkv, max_k), -7, dtype=torch.int32, device=dev)
            keep_new = torch.full((L, B, Hkv, max_k), -9, dtype=torch.int32, device=dev)
            ctx.rasr_prune(ref, bud, 32, 4, keep_ref)
            st_ref, item_ref = ctx.poll_status()
            status = torch.full((2,), 77, dtype=torch.int32, device=dev)
            torch.cuda.synchronize()
            free_before = _free_bytes()
            rc = binding.rasr_prune_static(new, bud, 32, 4, keep_new, status)
            assert rc == binding.OK
            torch.cuda.synchronize()
            if rnd > 0:                                        # the first call on a device may load the library image
                assert _free_bytes() == free_before, "the call changed the device's free memory"
            st_o, keep_o = oracle.rasr_prune(oc, budgets, 32, 4, max_k=max_k)
            # the status code must agree; which of several offending items reports first is a race on both sides
            assert status.tolist()[0] == st_ref == (binding.ERR_BUDGET if st_o == oracle.ERR_BUDGET else 0), \
                (rnd, status.tolist(), st_ref, item_ref, st_o)
            assert torch.equal(keep_new.cpu(), keep_o), f"round {rnd}: kept slots differ from the oracle's"
            assert torch.equal(keep_new, keep_ref), f"round {rnd}: kept slots differ from lethe_rasr_prune's"
            assert_state_matches(new, oc, exact_rel=True)      # len, pos, rel and the moved K / V rows: bit-exact
            assert_state_matches(ref, oc, exact_rel=True)
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
