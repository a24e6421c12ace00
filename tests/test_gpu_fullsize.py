"""Parity at the full size of the Llama-8B-shaped workload (the one bench.py times), of the Qwen-7B-shaped one and of
the long-reasoning stress shape,
in exactly the launch configuration bench.py uses (its Runner: all layers x sequences x KV heads in one
lethe_decode_attend call, default tuning).  The oracle cannot run the whole state in seconds, so it recomputes
sampled items one by one from snapshots of the GPU state taken just before the call."""
import pytest
import torch

import oracle
from helpers import gpu_context

pytestmark = pytest.mark.gpu


def _item_cache(k, v, rel, pos, n, G, D, cap):
    """Single-item OracleCache (1 layer, 1 sequence, 1 KV head, G query heads)."""
    return oracle.OracleCache(1, 1, G, 1, D, cap, k.reshape(1, 1, 1, cap, D).contiguous(),
                              v.reshape(1, 1, 1, cap, D).contiguous(), rel.reshape(1, 1, 1, cap).contiguous(),
                              pos.reshape(1, 1, 1, cap).contiguous(), torch.tensor([[[n]]], dtype=torch.int32))


@pytest.mark.parametrize("name,cap_factor", [("llama8b", 2), ("qwen7b", 3), ("longreason", 3)])
def test_full_size_sampled_items(name, cap_factor):
    import bench
    from paper_2511_06029_b200 import synth
    gpu_context().close()                          # builds the library if needed
    w = synth.WORKLOADS[name]
    dev = torch.device("cuda", 0)
    cap = cap_factor * w.mean_budget
    r = bench.Runner(w, dev, 0, cap, 0, 0)
    for _ in range(w.prune_interval):               # one prep round, as bench.py does
        r.decode()
    r.prune()
    for _ in range(5):
        r.decode()
    r.check()
    c = r.cache
    L, B, H, G, D = w.n_layers, w.batch, w.n_kv_heads, w.group, w.head_dim
    lens = c.len.cpu()
    flat = lens.flatten()
    g = torch.Generator().manual_seed(0)
    picks = set(torch.randint(0, flat.numel(), (8,), generator=g).tolist())
    picks |= {int(flat.argmax()), int(flat.argmin()), 0, flat.numel() - 1}
    picks = sorted(picks)

    # ---- one decode step: snapshot sampled items, run the full launch, recompute the samples on the CPU
    snaps = {}
    for it in picks:
        l, b, h = it // (B * H), (it // H) % B, it % H
        snaps[it] = tuple(t[l, b, h].cpu().clone() for t in (c.k, c.v, c.rel, c.pos))
    q, kn, vn = r.pool[r.step_no % len(r.pool)]
    r.decode()
    r.check()
    out = r.out.cpu()
    scale = synth.layer_scales(w)
    for it in picks:
        l, b, h = it // (B * H), (it // H) % B, it % H
        k0, v0, rel0, pos0 = snaps[it]
        n = int(lens[l, b, h])
        oc = _item_cache(k0, v0, rel0, pos0, n, G, D, cap)
        sc = torch.full((1,), float(scale[l]))
        st, o_ref, _, _ = oracle.decode_attend(oc, 0, 1, q[l, b, h * G:(h + 1) * G].cpu().reshape(1, 1, G, D).contiguous(),
                                               kn[l, b, h].cpu().reshape(1, 1, 1, D).contiguous(),
                                               vn[l, b, h].cpu().reshape(1, 1, 1, D).contiguous(),
                                               r.token_pos[b:b + 1].cpu(), sc, w.gamma)
        assert st == oracle.OK
        err = (out[l, b, h * G:(h + 1) * G].double() - o_ref[0, 0].double()).abs().max().item()
        assert err <= 2e-2, (it, err)
        assert int(c.len[l, b, h]) == n + 1
        assert torch.allclose(c.rel[l, b, h, :n + 1].cpu(), oc.rel[0, 0, 0, :n + 1], rtol=1e-3, atol=1e-6), it
        assert torch.equal(c.k[l, b, h, :n + 1].cpu().view(torch.int16), oc.k[0, 0, 0, :n + 1].view(torch.int16))
        assert torch.equal(c.v[l, b, h, n].cpu().view(torch.int16), oc.v[0, 0, 0, n].view(torch.int16))
        assert torch.equal(c.pos[l, b, h, :n + 1].cpu(), oc.pos[0, 0, 0, :n + 1])

    # ---- one prune round: sparsity and budgets of two whole sequences, retention of sampled items
    while not r.prune_due():
        r.decode()
    r.check()
    lens = c.len.cpu()
    seqs = [1, B - 1]
    rel_seq = {b: c.rel[:, b].cpu().clone() for b in seqs}
    snaps = {}
    items = [(l, b, h) for b in seqs for (l, h) in [(0, 0), (7, 3 % H), (19, 5 % H), (L - 1, H - 1)]]
    for (l, b, h) in items:
        snaps[(l, b, h)] = tuple(t[l, b, h].cpu().clone() for t in (c.k, c.v, c.rel, c.pos))
    r.prune()
    r.check()
    S = r.S.cpu(); bud = r.budgets.cpu()
    for b in seqs:
        dummy = torch.zeros((L, 1, H, 1, 1), dtype=torch.bfloat16)
        oc = oracle.OracleCache(L, 1, w.n_q_heads, H, 1, cap, dummy, dummy, rel_seq[b].reshape(L, 1, H, cap).contiguous(),
                                torch.zeros((L, 1, H, cap), dtype=torch.int32), lens[:, b].reshape(L, 1, H).contiguous())
        # estimate_sparsity reads only rel and len
        st, S_ref = oracle.estimate_sparsity(oc)
        assert st == oracle.OK and torch.allclose(S[:, b], S_ref[:, 0], rtol=1e-3, atol=1e-6)
        st, bud_ref = oracle.alloc_budgets(S[:, b:b + 1].contiguous(), torch.tensor([w.total_budget], dtype=torch.int64), w.k_min)
        assert st == oracle.OK and torch.equal(bud[:, b], bud_ref[:, 0])       # bit-exact given the same fp32 sparsity
        assert int(bud[:, b].sum()) == w.total_budget
    for (l, b, h) in items:
        k0, v0, rel0, pos0 = snaps[(l, b, h)]
        n = int(lens[l, b, h])
        oc = _item_cache(k0, v0, rel0, pos0, n, G, D, cap)
        st, keep = oracle.rasr_prune(oc, bud[l:l + 1, b:b + 1].contiguous(), w.recent, w.sink, max_k=cap)
        assert st == oracle.OK
        m = int(oc.len[0, 0, 0])
        assert int(c.len[l, b, h]) == m == min(n, int(bud[l, b]))
        for name, ref in (("k", oc.k), ("v", oc.v), ("rel", oc.rel), ("pos", oc.pos)):
            got = getattr(c, name)[l, b, h, :m].cpu()
            assert torch.equal(got.view(torch.uint8), ref[0, 0, 0, :m].view(torch.uint8)), (name, l, b, h)
    # properties that hold at any size
    lens_after = c.len.cpu()
    assert torch.all(lens_after <= torch.minimum(lens, bud[:, :, None].expand(L, B, H)))
    r.ctx.close()
    del r, c
    torch.cuda.empty_cache()
