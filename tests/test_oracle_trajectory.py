"""The oracle on whole workloads: the Tiny configuration end to end with every invariant checked at every
step, and the paged layout against the contiguous one."""
import math

import torch

import oracle
from helpers import cache_from_state, oracle_prune_round
from paper_2511_06029_b200 import synth


def test_tiny_trajectory_invariants():
    w = synth.WORKLOADS["tiny"]
    cap = w.prompt_len + w.prune_interval
    for sink in (w.sink, 0):
        state = synth.initial_kv(w, w.prompt_len, cap)
        c = cache_from_state(w, state, cap)
        scale = synth.layer_scales(w)
        T = torch.tensor([w.total_budget], dtype=torch.int64)
        expected_len = w.prompt_len
        mass_total = torch.zeros((w.n_layers, 1, w.n_kv_heads), dtype=torch.float64)
        for step in range(w.gen_steps):
            x = synth.step_inputs(w, step)
            prev_pos = c.pos.clone()
            st, out, lse, probs = oracle.decode_attend(c, 0, 1, x["q"], x["k_new"], x["v_new"], x["token_pos"], scale,
                                                       w.gamma, want_lse=True, want_probs=True)
            assert st == oracle.OK
            expected_len += 1
            assert torch.all(c.len == expected_len)
            n = expected_len
            assert torch.allclose(probs[..., :n].sum(-1), torch.ones((1, 1, w.n_q_heads), dtype=torch.float64), atol=1e-12)
            assert torch.all(c.pos[..., n - 1] == w.prompt_len + step)
            assert torch.all(torch.isfinite(out))
            # each step adds exactly G units of attention mass to every KV head's relevance (Eq. 5)
            mass_total = w.gamma * mass_total + w.group
            assert torch.allclose(c.rel[..., :n].double().sum(-1), mass_total, rtol=1e-5)
            if (step + 1) % w.prune_interval == 0:
                before = c.clone()
                st, S, budgets, keep = oracle_prune_round(c, T, sink + w.recent, w.recent, sink, max_k=cap)
                assert st == oracle.OK
                assert torch.all((S >= 0) & (S <= 1))
                assert int(budgets.sum()) == w.total_budget            # one layer: the whole budget
                k = int(budgets[0, 0])
                for h in range(w.n_kv_heads):
                    kept = [i for i in keep[0, 0, h].tolist() if i >= 0]
                    assert len(kept) == k == int(c.len[0, 0, h])         # each head keeps exactly its budget
                    assert set(range(sink)) <= set(kept)
                    assert set(range(n - w.recent, n)) <= set(kept)      # recent window always kept
                    dropped = sorted(set(range(sink, n - w.recent)) - set(kept))
                    chosen = sorted(set(kept) - set(range(sink)) - set(range(n - w.recent, n)))
                    if dropped and chosen:
                        r = before.rel[0, 0, h]
                        assert r[chosen].min() >= r[dropped].max()
                    idx = torch.tensor(kept)
                    assert torch.equal(c.k[0, 0, h, :k], before.k[0, 0, h, idx])
                    assert torch.equal(c.pos[0, 0, h, :k], before.pos[0, 0, h, idx])
                    assert torch.all(c.pos[0, 0, h, 1:k] > c.pos[0, 0, h, :k - 1])
                expected_len = k
                mass_total = c.rel[..., :k].double().sum(-1)
        assert expected_len == w.total_budget


def test_anchors_attract_relevance_in_tiny():
    """Sanity of the workload itself: after the first prune of Tiny the scaled-key anchors are over-represented
    among retained prompt tokens (the synthetic stand-in for 'salient' tokens)."""
    w = synth.WORKLOADS["tiny"]
    cap = w.prompt_len + w.prune_interval
    state = synth.initial_kv(w, w.prompt_len, cap)
    c = cache_from_state(w, state, cap)
    flags = synth.anchor_flags(w, torch.arange(w.prompt_len), torch.arange(1))[0, 0]
    assert int(flags.sum()) == 16
    for step in range(w.prune_interval):
        x = synth.step_inputs(w, step)
        oracle.decode_attend(c, 0, 1, x["q"], x["k_new"], x["v_new"], x["token_pos"], synth.layer_scales(w), w.gamma)
    oracle_prune_round(c, torch.tensor([w.total_budget], dtype=torch.int64), w.k_min, w.recent, w.sink)
    kept_pos = c.pos[0, 0, 0, :int(c.len[0, 0, 0])].long()
    kept_prompt = kept_pos[kept_pos < w.prompt_len]
    frac_anchor_kept = flags[kept_prompt].float().mean().item()
    assert frac_anchor_kept > 3 * 16 / w.prompt_len


def test_paged_equals_contiguous():
    """Same logical content in 16-token pages behind a shuffled page table: every call gives identical
    results and identical logical state."""
    w = synth.shrink(synth.WORKLOADS["ragged"], n_layers=2, batch=2, n_q_heads=14, n_kv_heads=2, head_dim=32,
                     prompt_len=70)
    cap = 96
    st_c = synth.initial_kv(w, 70, cap)
    # ragged lengths
    st_c["len"][0, 0, 0] = 33; st_c["len"][1, 1, 1] = 16; st_c["len"][1, 0, 0] = 1
    st_p = synth.to_paged({k: v.clone() for k, v in st_c.items()}, 16, seed=3, spare_pages=5)
    cc = cache_from_state(w, st_c, cap); cp = cache_from_state(w, st_p, cap)
    scale = synth.layer_scales(w)
    T = torch.tensor([60, 90], dtype=torch.int64)

    def logical(c):
        L, B, H = c.len.shape
        rows = []
        for l in range(L):
            for b in range(B):
                for h in range(H):
                    n = int(c.len[l, b, h])
                    if c.paged:
                        pg = c.page_table[l, b, h].long()
                        kk = c.k[pg].reshape(-1, c.head_dim)[:n]; vv = c.v[pg].reshape(-1, c.head_dim)[:n]
                    else:
                        kk = c.k[l, b, h, :n]; vv = c.v[l, b, h, :n]
                    rows.append((kk.clone(), vv.clone(), c.rel[l, b, h, :n].clone(), c.pos[l, b, h, :n].clone()))
        return rows

    for step in range(6):
        x = synth.step_inputs(w, step)
        a = oracle.decode_attend(cc, 0, 2, x["q"], x["k_new"], x["v_new"], x["token_pos"], scale, 0.9, want_lse=True)
        b = oracle.decode_attend(cp, 0, 2, x["q"], x["k_new"], x["v_new"], x["token_pos"], scale, 0.9, want_lse=True)
        assert a[0] == b[0] == oracle.OK and torch.equal(a[1], b[1]) and torch.equal(a[2], b[2])
        if step in (2, 5):
            ra = oracle_prune_round(cc, T, 6, 5, 1, max_k=cap)
            rb = oracle_prune_round(cp, T, 6, 5, 1, max_k=cap)
            assert ra[0] == rb[0] and torch.equal(ra[1], rb[1]) and torch.equal(ra[2], rb[2]) and torch.equal(ra[3], rb[3])
        assert torch.equal(cc.len, cp.len)
        for ra_, rb_ in zip(logical(cc), logical(cp)):
            for u, v_ in zip(ra_, rb_):
                assert torch.equal(u, v_)


def test_long_reasoning_anchor_drift_is_a_real_redraw():
    """The long-reasoning workload re-draws its anchor positions every 2048 decode steps: the sets of two epochs
    are independent draws of the same density over ALL positions (old tokens included), the token generated at a
    step is an anchor by the draw in force at that step, and re-drawing a cache rescales exactly the K rows whose
    flag changed (by the anchor gain or its inverse), wherever pruning has moved them."""
    from paper_2511_06029_b200 import synth
    w = synth.shrink(synth.WORKLOADS["longreason"], n_layers=2, batch=3)
    assert synth.drift_epoch(w, 0) == 0 and synth.drift_epoch(w, 2047) == 0 and synth.drift_epoch(w, 2048) == 1
    pos = torch.arange(20000)
    f0 = synth.anchor_flags(w, pos, torch.arange(3), 0)
    f1 = synth.anchor_flags(w, pos, torch.arange(3), 1)
    for f in (f0, f1):
        assert 0.007 < f.float().mean() < 0.013                      # Bernoulli(1 %)
    assert (f0 & f1).float().mean() < 0.0005                         # independent: overlap ~ 1e-4
    assert torch.equal(f0[0], f0[1])                                 # shared across layers (per-sequence rule)
    # a cache whose slots hold a shuffled subset of positions (as after pruning)
    st = synth.initial_kv(w, 600, 608)
    g = torch.Generator().manual_seed(3)
    keep = torch.sort(torch.randperm(600, generator=g)[:200]).values
    for key in ("k", "v"):
        st[key][..., :200, :] = st[key][..., keep, :]
    st["pos"][..., :200] = keep.to(torch.int32)
    st["len"][:] = 200
    k0 = st["k"].clone()
    synth.apply_drift(w, st["k"], st["pos"], torch.arange(3), 0, 1)
    ratio = (st["k"].float().norm(dim=-1) / k0.float().norm(dim=-1))[..., :200]
    fl0 = synth.anchor_flags(w, keep, torch.arange(3), 0)[:, :, None, :].expand_as(ratio)
    fl1 = synth.anchor_flags(w, keep, torch.arange(3), 1)[:, :, None, :].expand_as(ratio)
    assert torch.allclose(ratio[fl1 & ~fl0], torch.tensor(3.0), rtol=2e-2)
    assert torch.allclose(ratio[fl0 & ~fl1], torch.tensor(1 / 3.0), rtol=2e-2)
    assert torch.equal(st["k"][..., :200, :][~(fl0 ^ fl1)], k0[..., :200, :][~(fl0 ^ fl1)])
    # the generated token of step 2048 + 5 follows epoch 1
    x = synth.step_inputs(w, 2053)
    p = w.prompt_len + 2053
    want = synth.anchor_flags(w, torch.tensor([p]), torch.arange(3), 1)[..., 0]            # [L][B]
    big = x["k_new"].float().norm(dim=-1).mean(dim=-1) > 1.8 * (w.head_dim ** 0.5)          # anchor rows are x3
    assert torch.equal(big, want)
