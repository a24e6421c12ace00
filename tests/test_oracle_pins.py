"""Pins for the CPU oracle: what the paper's definitions and plain mathematics fix, checked without a GPU.

Each test is chosen so that a plausible slip in the oracle (dropped term, wrong sign or index, transposed
operand, wrong head grouping, wrong tie order) makes it fail.
"""
import itertools
import json
import math
import os
from fractions import Fraction

import pytest
import torch

import oracle
from helpers import random_cache

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "closed_forms.json")))


def _scale(L, val):
    return torch.full((L,), val, dtype=torch.float32)


# --------------------------------------------------------------------------- attention (Sec. 4.2, Eq. 3)

def test_golden_attention_and_relevance():
    g = GOLD["attention"]
    k = torch.tensor([[math.log(a), c] for a, c in zip(g["k_ln_of"], g["k_second_col"])], dtype=torch.float32)
    v = torch.tensor(g["v"], dtype=torch.float32)
    cap = 4
    K = torch.zeros((1, 1, 1, cap, 2)); V = torch.zeros((1, 1, 1, cap, 2))
    K[0, 0, 0, :3] = k; V[0, 0, 0, :3] = v
    c = oracle.OracleCache(1, 1, 2, 1, 2, cap, K, V, torch.zeros((1, 1, 1, cap)),
                           torch.zeros((1, 1, 1, cap), dtype=torch.int32), torch.tensor([[[3]]], dtype=torch.int32))
    q = torch.tensor(g["q"], dtype=torch.float32).reshape(1, 1, 2, 2)
    st, out, lse, probs = oracle.decode_attend(c, 0, 1, q, None, None, None, _scale(1, g["scale"]), 0.9,
                                               want_lse=True, want_probs=True)
    assert st == oracle.OK
    assert torch.allclose(probs[0, 0, :, :3], torch.tensor(g["p"], dtype=torch.float64), atol=1e-7)
    assert torch.allclose(out[0, 0].double(), torch.tensor(g["o"], dtype=torch.float64), atol=1e-5)
    assert torch.allclose(c.rel[0, 0, 0, :3].double(), torch.tensor(g["rel_step1"], dtype=torch.float64), atol=1e-6)
    assert abs(lse[0, 0, 0].item() - math.log(7.0)) < 1e-6 and abs(lse[0, 0, 1].item() - math.log(3.0)) < 1e-6
    st, _, _, _ = oracle.decode_attend(c, 0, 1, q, None, None, None, _scale(1, g["scale"]), g["gamma2"])
    assert torch.allclose(c.rel[0, 0, 0, :3].double(), torch.tensor(g["rel_step2"], dtype=torch.float64), atol=1e-6)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("Hq,Hkv", [(8, 2), (7, 1), (4, 4)])
def test_attention_matches_library_sdpa(dtype, Hq, Hkv):
    """Special case that reduces to a library routine: fp64 SDPA on K/V expanded per query head (Eq. 3's
    `repeat`), with a different length for every item."""
    L, B, D, cap = 2, 3, 16, 40
    lens = torch.randint(1, cap + 1, (L, B, Hkv), generator=torch.Generator().manual_seed(5))
    c = random_cache(L, B, Hq, Hkv, D, cap, lens, dtype=dtype, seed=11)
    g = torch.Generator().manual_seed(3)
    q = torch.randn((L, B, Hq, D), generator=g).to(dtype)
    scale = torch.tensor([0.37, 0.11], dtype=torch.float32)
    st, out, lse, probs = oracle.decode_attend(c, 0, L, q, None, None, None, scale, 0.5, want_lse=True,
                                               want_probs=True)
    assert st == oracle.OK
    G = Hq // Hkv
    for l in range(L):
        for b in range(B):
            for h in range(Hq):
                n = int(lens[l, b, h // G])
                kk = c.k[l, b, h // G, :n].double(); vv = c.v[l, b, h // G, :n].double()
                ref = torch.nn.functional.scaled_dot_product_attention(
                    q[l, b, h].double()[None, None, None, :], kk[None, None], vv[None, None],
                    scale=float(scale[l]))[0, 0, 0]
                tol = 1e-6 if dtype == torch.float32 else 1.6e-2   # bf16: one rounding of |o| < 4 is <= 2^-7
                assert torch.allclose(out[l, b, h].double(), ref, atol=tol), (l, b, h)
                s = (kk @ q[l, b, h].double()) * float(scale[l])
                assert abs(lse[l, b, h].item() - torch.logsumexp(s, 0).item()) < 1e-5
                assert abs(probs[l, b, h, :n].sum().item() - 1.0) < 1e-12          # softmax rows sum to one
                assert torch.all(probs[l, b, h, n:] == 0)
                # relevance from zero equals the group's summed library softmax (Eq. 5 with s_0 = 0)
    for l in range(L):
        for b in range(B):
            for hk in range(Hkv):
                n = int(lens[l, b, hk])
                kk = c.k[l, b, hk, :n].double()
                mass = torch.zeros(n, dtype=torch.float64)
                for g_ in range(G):
                    mass += torch.softmax((kk @ q[l, b, hk * G + g_].double()) * float(scale[l]), 0)
                assert torch.allclose(c.rel[l, b, hk, :n].double(), mass, rtol=1e-6, atol=1e-8)
                assert torch.all(c.rel[l, b, hk, n:] == 0)


def test_uniform_attention_closed_forms():
    """q = 0 gives p = 1/n and o = column mean of V; n = 1 gives o = V[0]."""
    c = random_cache(1, 1, 4, 2, 8, 16, torch.tensor([[[9, 1]]]), seed=2)
    q = torch.zeros((1, 1, 4, 8))
    q[0, 0, 2:] = torch.randn((2, 8), generator=torch.Generator().manual_seed(1))   # heads of the n = 1 item
    st, out, _, probs = oracle.decode_attend(c, 0, 1, q, None, None, None, _scale(1, 0.3), 0.9, want_probs=True)
    assert torch.allclose(probs[0, 0, 0, :9], torch.full((9,), 1 / 9, dtype=torch.float64), atol=1e-15)
    assert torch.allclose(out[0, 0, 0], c.v[0, 0, 0, :9].mean(0), atol=1e-6)
    assert torch.equal(out[0, 0, 2], c.v[0, 0, 1, 0]) and torch.equal(out[0, 0, 3], c.v[0, 0, 1, 0])


def test_append_semantics():
    """The new token is written at slot len, gets pos = token_pos, starts at zero relevance and attends to
    itself in the same step (Sec. 4.1)."""
    c = random_cache(1, 2, 4, 2, 8, 8, 5, seed=4, rel_init="rand")
    before = c.clone()
    g = torch.Generator().manual_seed(9)
    q = torch.randn((1, 2, 4, 8), generator=g); kn = torch.randn((1, 2, 2, 8), generator=g)
    vn = torch.randn((1, 2, 2, 8), generator=g)
    tp = torch.tensor([100, 200], dtype=torch.int32)
    st, out, _, probs = oracle.decode_attend(c, 0, 1, q, kn, vn, tp, _scale(1, 0.35), 0.75, want_probs=True)
    assert st == oracle.OK
    assert torch.all(c.len == 6)
    assert torch.equal(c.k[0, :, :, 5], kn[0]) and torch.equal(c.v[0, :, :, 5], vn[0])
    assert torch.equal(c.k[0, :, :, :5], before.k[0, :, :, :5])
    assert torch.all(c.pos[0, 0, :, 5] == 100) and torch.all(c.pos[0, 1, :, 5] == 200)
    for b in range(2):
        for hk in range(2):
            mass = probs[0, b, 2 * hk:2 * hk + 2, :6].sum(0)
            want = 0.75 * before.rel[0, b, hk, :6].double() + mass
            want[5] = mass[5]                       # new token: zero history
            assert torch.allclose(c.rel[0, b, hk, :6].double(), want, rtol=1e-6)
            assert mass[5] > 0
    # a full cache refuses the append and changes nothing
    full = random_cache(1, 1, 2, 1, 4, 3, 3, seed=1)
    snap = full.clone()
    st, *_ = oracle.decode_attend(full, 0, 1, torch.zeros((1, 1, 2, 4)), torch.ones((1, 1, 1, 4)),
                                  torch.ones((1, 1, 1, 4)), torch.tensor([7], dtype=torch.int32), _scale(1, 1.0), 0.9)
    assert st == oracle.ERR_CAPACITY
    assert torch.equal(full.k, snap.k) and torch.equal(full.len, snap.len)


# --------------------------------------------------------------------------- relevance recurrence (Eq. 5)

@pytest.mark.parametrize("gamma", [0.5, 0.9, 1.0])
def test_relevance_mass_conservation(gamma):
    """Without pruning every step adds exactly G (one unit of attention per query head), so from zero
    sum_j rel_t = G (1 - gamma^t)/(1 - gamma), or G t when gamma = 1."""
    L, B, Hq, Hkv, D, cap = 1, 2, 6, 2, 8, 24
    G = Hq // Hkv
    c = random_cache(L, B, Hq, Hkv, D, cap, 4, seed=8)
    g = torch.Generator().manual_seed(21)
    for t in range(1, 13):
        q = torch.randn((L, B, Hq, D), generator=g); kn = torch.randn((L, B, Hkv, D), generator=g)
        vn = torch.randn((L, B, Hkv, D), generator=g)
        st, *_ = oracle.decode_attend(c, 0, L, q, kn, vn, torch.full((B,), t, dtype=torch.int32), _scale(L, 0.4),
                                      gamma)
        assert st == oracle.OK
        want = G * t if gamma == 1.0 else G * (1 - gamma ** t) / (1 - gamma)
        tot = c.rel.double().sum(-1)
        assert torch.allclose(tot, torch.full_like(tot, want), rtol=1e-5)


def test_relevance_linearity_in_history():
    """rel after a block of steps = gamma^steps * (history) + (the same block run from zero history)."""
    mk = lambda init: random_cache(1, 1, 4, 2, 8, 12, 12, seed=3, rel_init=init)
    a, z = mk("rand"), mk("zero")
    hist = a.rel.clone()
    g = torch.Generator().manual_seed(2)
    gamma, steps = 0.8, 5
    for _ in range(steps):
        q = torch.randn((1, 1, 4, 8), generator=g)
        oracle.decode_attend(a, 0, 1, q, None, None, None, _scale(1, 0.5), gamma)
        oracle.decode_attend(z, 0, 1, q, None, None, None, _scale(1, 0.5), gamma)
    assert torch.allclose(a.rel.double(), gamma ** steps * hist.double() + z.rel.double(), rtol=2e-6, atol=1e-7)


# --------------------------------------------------------------------------- Hoyer sparsity (Eq. 1)

def _hoyer_cache(vectors, cap=None):
    """One layer, one sequence, one KV head per vector."""
    H = len(vectors)
    cap = cap or max(len(v) for v in vectors)
    rel = torch.zeros((1, 1, H, cap))
    ln = torch.zeros((1, 1, H), dtype=torch.int32)
    for i, v in enumerate(vectors):
        rel[0, 0, i, :len(v)] = torch.tensor(v, dtype=torch.float32)
        ln[0, 0, i] = len(v)
    z = torch.zeros((1, 1, H, cap, 2))
    return oracle.OracleCache(1, 1, H, H, 2, cap, z, z.clone(), rel, torch.zeros((1, 1, H, cap), dtype=torch.int32), ln)


def test_golden_hoyer():
    for case in GOLD["hoyer"]:
        st, s = oracle.estimate_sparsity(_hoyer_cache([case["a"]]))
        assert st == oracle.OK and abs(s.item() - case["expect"]) < 1e-6, case


def test_hoyer_properties():
    g = torch.Generator().manual_seed(0)
    for n in (2, 3, 17, 100):
        a = torch.rand(n, generator=g).tolist()
        s1 = oracle.estimate_sparsity(_hoyer_cache([a]))[1].item()
        s2 = oracle.estimate_sparsity(_hoyer_cache([[x * 37.5 for x in a]]))[1].item()
        assert 0.0 <= s1 <= 1.0 and abs(s1 - s2) < 1e-6                      # range, scale invariance
        for m in range(1, n + 1):                                            # m equal non-zeros of n
            vec = [2.5] * m + [0.0] * (n - m)
            want = (math.sqrt(n) - math.sqrt(m)) / (math.sqrt(n) - 1)
            assert abs(oracle.estimate_sparsity(_hoyer_cache([vec]))[1].item() - want) < 1e-6
    # degenerate: length 0 or 1, zero vector -> 0; slots beyond len are ignored
    c = _hoyer_cache([[5.0], [0.0, 0.0, 0.0], [1.0, 1.0]], cap=6)
    c.rel[0, 0, 2, 2:] = 99.0
    assert abs(oracle.estimate_sparsity(c)[1].item()) < 1e-12
    # layer value = mean over the KV heads
    c = _hoyer_cache([[1.0, 0, 0, 0], [1.0, 1, 1, 1], [1.0, 1, 0, 0]])
    assert abs(oracle.estimate_sparsity(c)[1].item() - (1 + 0 + (2 - math.sqrt(2))) / 3) < 1e-6


# --------------------------------------------------------------------------- budgets (Sec. 4.2)

def _lr_fraction(S, T, k_min):
    """Exact-rational largest-remainder apportionment of the weights the rule defines."""
    w = []
    for s in S:
        s32 = torch.tensor(s, dtype=torch.float32)
        s32 = torch.where(s32 >= 0, s32, torch.zeros(())).clamp(max=1.0) if not math.isnan(s) else torch.zeros(())
        d = (torch.tensor(1.0, dtype=torch.float32) - s32)
        w.append(max(1, int(torch.round(d * 1048576.0).item())))
    F = T - len(S) * k_min
    W = sum(w)
    quota = [Fraction(wi * F, W) for wi in w]
    base = [q.numerator // q.denominator for q in quota]
    order = sorted(range(len(S)), key=lambda i: (-(quota[i] - base[i]), i))
    for i in order[:F - sum(base)]:
        base[i] += 1
    return [k_min + x for x in base]


def test_golden_budgets():
    for case in GOLD["budgets"]:
        S = torch.tensor(case["sparsity"], dtype=torch.float32)[:, None]
        st, k = oracle.alloc_budgets(S, torch.tensor([case["total"]], dtype=torch.int64), case["k_min"])
        assert st == oracle.OK and k[:, 0].tolist() == case["expect"], case


def test_budget_invariants_and_exact_rationals():
    g = torch.Generator().manual_seed(7)
    for trial in range(60):
        L = int(torch.randint(1, 40, (1,), generator=g)); B = int(torch.randint(1, 5, (1,), generator=g))
        S = torch.rand((L, B), generator=g)
        if trial % 5 == 0:
            S[0] = float("nan"); S[-1] = 1.0
        if trial % 7 == 0:
            S[:] = S[0, 0]                                       # all equal
        k_min = int(torch.randint(0, 70, (1,), generator=g))
        T = torch.randint(L * k_min, L * k_min + 5000, (B,), generator=g, dtype=torch.int64)
        st, k = oracle.alloc_budgets(S, T, k_min)
        assert st == oracle.OK
        assert torch.equal(k.long().sum(0), T)                   # layer budgets sum to the global budget
        assert torch.all(k >= k_min)
        for b in range(B):
            assert k[:, b].tolist() == _lr_fraction(S[:, b].tolist(), int(T[b]), k_min)
            Sb = torch.nan_to_num(S[:, b], nan=0.0)
            for i in range(L):                                   # sparser layer never gets more
                for j in range(L):
                    if Sb[i] > Sb[j]:
                        assert k[i, b] <= k[j, b]
        if trial % 7 == 0:
            F = T - L * k_min
            for b in range(B):
                want = [k_min + int(F[b]) // L + (1 if l < int(F[b]) % L else 0) for l in range(L)]
                assert k[:, b].tolist() == want
    st, _ = oracle.alloc_budgets(torch.zeros((4, 1)), torch.tensor([39], dtype=torch.int64), 10)
    assert st == oracle.ERR_BUDGET


# --------------------------------------------------------------------------- selection and compaction

def _prune_one(rel, k, recent, sink, D=4, seed=0):
    n = len(rel)
    c = random_cache(1, 1, 1, 1, D, n + 3, n, seed=seed)
    c.rel[0, 0, 0, :n] = torch.tensor(rel, dtype=torch.float32)
    before = c.clone()
    st, keep = oracle.rasr_prune(c, torch.tensor([[k]], dtype=torch.int32), recent, sink, max_k=n + 3)
    kept = [i for i in keep[0, 0, 0].tolist() if i >= 0]
    return st, kept, c, before


def test_golden_select():
    g = GOLD["select"]
    st, kept, c, before = _prune_one(g["rel"], g["budget"], g["recent"], g["sink"])
    assert st == oracle.OK and kept == g["expect"]


def test_select_brute_force_tiny():
    """n <= 11: among all size-k supersets of the protected set, the kept set has the largest score sum and,
    among those, the lexicographically smallest index tuple."""
    g = torch.Generator().manual_seed(13)
    for trial in range(120):
        n = int(torch.randint(2, 12, (1,), generator=g))
        sink = int(torch.randint(0, 3, (1,), generator=g)); recent = int(torch.randint(0, 4, (1,), generator=g))
        # few distinct values -> many ties
        rel = (torch.randint(0, 4, (n,), generator=g).float() * 0.25).tolist()
        prot = set(range(min(sink, n))) | set(range(n - min(recent, n), n))
        if len(prot) >= n:
            continue
        k = int(torch.randint(len(prot), n, (1,), generator=g))
        st, kept, _, _ = _prune_one(rel, k, recent, sink, seed=trial)
        assert st == oracle.OK and len(kept) == k and prot <= set(kept)
        rest = [j for j in range(n) if j not in prot]
        best = None
        for extra in itertools.combinations(rest, k - len(prot)):
            key = (-sum(rel[j] for j in extra), tuple(sorted(extra)))
            if best is None or key < best:
                best = key
        assert tuple(sorted(set(kept) - prot)) == best[1], (rel, k, sink, recent, kept)


def test_select_matches_stable_sort_and_compaction_is_a_gather():
    g = torch.Generator().manual_seed(17)
    for n, k, recent, sink in [(300, 100, 32, 4), (4096, 1000, 64, 4), (1000, 999, 0, 0), (513, 36, 32, 4),
                               (200, 50, 0, 7), (200, 50, 9, 0)]:
        rel = torch.rand(n, generator=g)
        rel[torch.randint(0, n, (n // 3,), generator=g)] = 0.5           # ties
        st, kept, c, before = _prune_one(rel.tolist(), k, recent, sink, D=8, seed=n)
        assert st == oracle.OK and len(kept) == k == int(c.len[0, 0, 0])
        cand = torch.arange(sink, n - recent)
        order = torch.sort(rel[cand], descending=True, stable=True).indices
        want = sorted(list(range(sink)) + list(range(n - recent, n)) + cand[order[:k - sink - recent]].tolist())
        assert kept == want
        idx = torch.tensor(kept)
        assert torch.equal(c.k[0, 0, 0, :k], before.k[0, 0, 0, idx]) and torch.equal(c.v[0, 0, 0, :k], before.v[0, 0, 0, idx])
        assert torch.equal(c.rel[0, 0, 0, :k], before.rel[0, 0, 0, idx]) and torch.equal(c.pos[0, 0, 0, :k], before.pos[0, 0, 0, idx])
        assert torch.all(c.pos[0, 0, 0, 1:k] > c.pos[0, 0, 0, :k - 1])


def test_select_special_cases():
    rel = torch.rand(50, generator=torch.Generator().manual_seed(1)).tolist()
    # budget >= length: bitwise identity (FullKV)
    for k in (50, 51, 1000):
        st, kept, c, before = _prune_one(rel, k, 8, 2)
        assert st == oracle.OK and kept == list(range(50))
        for name in ("k", "v", "rel", "pos", "len"):
            assert torch.equal(getattr(c, name), getattr(before, name))
    # budget = sink + recent: sinks plus window whatever the scores (StreamingLLM)
    st, kept, _, _ = _prune_one(rel, 10, 8, 2)
    assert kept == [0, 1] + list(range(42, 50))
    # all scores equal: the oldest candidates survive (tie order made visible)
    st, kept, _, _ = _prune_one([0.0] * 50, 15, 8, 2)
    assert kept == list(range(7)) + list(range(42, 50))
    # protected set larger than the budget: exactly the protected set, flagged
    st, kept, c, _ = _prune_one(rel, 5, 8, 2)
    assert st == oracle.ERR_BUDGET and kept == [0, 1] + list(range(42, 50)) and int(c.len[0, 0, 0]) == 10
    # sink and recent overlap (n < sink + recent): nothing to drop beyond the union
    st, kept, _, _ = _prune_one(rel[:6], 3, 4, 4)
    assert st == oracle.ERR_BUDGET and kept == list(range(6))


def test_multi_item_budgets_are_per_layer_and_sequence():
    L, B, Hkv = 3, 2, 2
    lens = torch.tensor([[[20, 25], [30, 18]], [[22, 22], [9, 40]], [[40, 40], [40, 40]]])
    c = random_cache(L, B, 4, Hkv, 4, 48, lens, seed=5, rel_init="rand")
    budgets = torch.tensor([[10, 20], [22, 12], [39, 40]], dtype=torch.int32)
    st, keep = oracle.rasr_prune(c, budgets, 3, 1, max_k=48)
    assert st == oracle.OK
    for l in range(L):
        for b in range(B):
            for h in range(Hkv):
                assert int(c.len[l, b, h]) == min(int(lens[l, b, h]), int(budgets[l, b]))
                kk = [i for i in keep[l, b, h].tolist() if i >= 0]
                assert len(kk) == int(c.len[l, b, h]) and kk == sorted(kk)


# --------------------------------------------------------------------------- Algorithm 1 (segmented breakpoint)

def _segment_one(rel, D, tau, recent, sink, l_evict, seed=0):
    n = len(rel)
    c = random_cache(1, 1, 1, 1, 4, n + 2, n, seed=seed)
    c.rel[0, 0, 0, :n] = torch.tensor(rel, dtype=torch.float32)
    before = c.clone()
    le = torch.tensor([[[l_evict]]], dtype=torch.int32)
    st, keep = oracle.segment_prune(c, D, tau, recent, sink, le, max_k=n + 2)
    kept = [i for i in keep[0, 0, 0].tolist() if i >= 0]
    return st, kept, int(le[0, 0, 0]), c, before


def test_golden_segment_prune():
    g = GOLD["segment"]
    st, kept, le, c, before = _segment_one(g["rel"], g["segments"], g["tau"], g["recent"], g["sink"], g["l_evict"])
    assert st == oracle.OK and kept == g["expect_keep"] and le == g["expect_l_evict"]
    idx = torch.tensor(kept)
    assert torch.equal(c.k[0, 0, 0, :len(kept)], before.k[0, 0, 0, idx]) and int(c.len[0, 0, 0]) == len(kept)
    nb = g["no_break"]
    st, kept, le, c, before = _segment_one(g["rel"], g["segments"], nb["tau"], g["recent"], g["sink"], g["l_evict"])
    assert kept == nb["expect_keep"] and le == nb["expect_l_evict"] and torch.equal(c.k, before.k)
    nt = g["not_triggered"]
    st, kept, le, c, before = _segment_one(g["rel"], g["segments"], g["tau"], g["recent"], g["sink"], nt["l_evict"])
    assert kept == list(range(8)) and le == nt["expect_l_evict"] and torch.equal(c.rel, before.rel)


def test_segment_prune_against_library_sort_and_invariants():
    """The sort step through torch.sort(stable=True); breakpoint, retention set and threshold update checked
    against the definitions; tau = 1 always breaks at the first cut, a huge tau never breaks."""
    g = torch.Generator().manual_seed(23)
    for trial in range(80):
        n = int(torch.randint(2, 400, (1,), generator=g)); D = int(torch.randint(2, 12, (1,), generator=g))
        sink = int(torch.randint(0, 5, (1,), generator=g)); recent = int(torch.randint(0, 40, (1,), generator=g))
        tau = [1.0, 1.5, 4.0, 50.0, 400.0, 1e30][trial % 6]
        rel = torch.rand(n, generator=g) ** 6                       # heavy-tailed scores
        rel[torch.randint(0, n, (n // 4,), generator=g)] = 0.125      # ties
        le0 = int(torch.randint(0, n + 5, (1,), generator=g))
        st, kept, le, c, before = _segment_one(rel.tolist(), D, tau, recent, sink, le0, seed=trial)
        assert st == oracle.OK
        if n <= le0:
            assert kept == list(range(n)) and le == le0
            continue
        order = torch.sort(rel, descending=True, stable=True)
        top_v, top_i = order.values, order.indices
        bp = -1
        for d in range(1, D):
            cpt = n * d // D
            if float(top_v[0]) >= float(torch.tensor(tau, dtype=torch.float32) * top_v[cpt]):
                bp = cpt; break
        if tau == 1.0:
            assert bp == n // D
        if tau == 1e30 and float(top_v[0]) > 0 and float(top_v[(n * 1) // D]) > 0:
            assert bp == -1
        if bp < 0:
            assert kept == list(range(n)) and le == min(2 * le0, 1 << 30) and torch.equal(c.k, before.k)
            continue
        prot = set(range(min(sink, n))) | set(range(max(0, n - recent), n))
        want = sorted(prot | set(top_i[:bp].tolist()))
        assert kept == want and le == max(le0, bp + recent)
        assert bp <= len(kept) <= bp + sink + recent
        idx = torch.tensor(kept)
        assert torch.equal(c.k[0, 0, 0, :len(kept)], before.k[0, 0, 0, idx]) and torch.equal(c.pos[0, 0, 0, :len(kept)], before.pos[0, 0, 0, idx])
        dropped = sorted(set(range(n)) - set(kept))
        salient = sorted(set(kept) - prot)
        if dropped and salient:
            assert rel[salient].min() >= rel[dropped].max()


# --------------------------------------------------------------------------- prefill seeding (Eq. 2 with Q > 1)

def test_prefill_seed_equals_token_by_token_decode():
    """Eq. 5 defines the relevance by a recurrence over steps; feeding the prompt one token at a time through the
    (separately pinned) decode step must leave exactly the scores that the prefill formula gives at once."""
    for dtype, Hq, Hkv, gamma in [(torch.float32, 4, 2, 0.9), (torch.bfloat16, 7, 1, 0.97), (torch.float32, 3, 3, 1.0)]:
        L, B, D, P, cap = 2, 2, 8, 21, 24
        g = torch.Generator().manual_seed(Hq)
        kk = torch.randn((L, B, Hkv, cap, D), generator=g).to(dtype); vv = torch.randn((L, B, Hkv, cap, D), generator=g).to(dtype)
        qp = torch.randn((L, B, P, Hq, D), generator=g).to(dtype)
        scale = torch.tensor([0.4, 0.15], dtype=torch.float32)
        mk = lambda n: oracle.OracleCache(L, B, Hq, Hkv, D, cap, kk.clone(), vv.clone(), torch.zeros((L, B, Hkv, cap)),
                                          torch.zeros((L, B, Hkv, cap), dtype=torch.int32),
                                          torch.full((L, B, Hkv), n, dtype=torch.int32))
        step = mk(0)
        for i in range(P):
            st, *_ = oracle.decode_attend(step, 0, L, qp[:, :, i].contiguous(), kk[:, :, :, i].contiguous(),
                                          vv[:, :, :, i].contiguous(), torch.full((B,), i, dtype=torch.int32), scale, gamma)
            assert st == oracle.OK
        once = mk(P)
        once.rel[:] = 123.0                                   # must be overwritten, not accumulated
        assert oracle.prefill_seed(once, qp, scale, gamma) == oracle.OK
        assert torch.allclose(once.rel[..., :P], step.rel[..., :P], rtol=2e-5, atol=1e-7)
        assert torch.all(once.rel[..., P:] == 123.0)


def test_prefill_seed_against_library_softmax_and_closed_forms():
    L, B, Hq, Hkv, D, P, cap = 1, 1, 4, 2, 16, 33, 40
    c = random_cache(L, B, Hq, Hkv, D, cap, P, seed=6)
    g = torch.Generator().manual_seed(4)
    qp = torch.randn((L, B, P, Hq, D), generator=g)
    scale = torch.tensor([0.3]); gamma = 0.8
    assert oracle.prefill_seed(c, qp, scale, gamma) == oracle.OK
    wgt = gamma ** torch.arange(P - 1, -1, -1, dtype=torch.float64)
    mask = torch.tril(torch.ones(P, P, dtype=torch.bool))
    for hk in range(Hkv):
        want = torch.zeros(P, dtype=torch.float64)
        for gq in range(2):
            s = (qp[0, 0, :, hk * 2 + gq].double() @ c.k[0, 0, hk, :P].double().T) * 0.3
            a = torch.softmax(s.masked_fill(~mask, float("-inf")), dim=1)
            want += (wgt[:, None] * a).sum(0)
        assert torch.allclose(c.rel[0, 0, hk, :P].double(), want, rtol=1e-6, atol=1e-9)
        # total mass: every prompt row hands out G units, decayed: G (1 - gamma^P) / (1 - gamma)
        assert abs(c.rel[0, 0, hk, :P].double().sum().item() - 2 * (1 - gamma ** P) / (1 - gamma)) < 1e-5
    # q = 0: row i spreads 1/(i+1) over slots 0..i
    c2 = random_cache(1, 1, 1, 1, 4, 8, 5, seed=1)
    assert oracle.prefill_seed(c2, torch.zeros((1, 1, 5, 1, 4)), torch.tensor([1.0]), 1.0) == oracle.OK
    want = torch.tensor([sum(1.0 / (i + 1) for i in range(j, 5)) for j in range(5)])
    assert torch.allclose(c2.rel[0, 0, 0, :5], want, atol=1e-6)
    short = random_cache(1, 1, 1, 1, 4, 8, 3, seed=1)
    assert oracle.prefill_seed(short, torch.zeros((1, 1, 5, 1, 4)), torch.tensor([1.0]), 1.0) == oracle.ERR_CAPACITY


# ----------------------------------------------------------------------------- collapsed score (Eq. 2 as printed)

def _collapsed_cache(rel, D=4, seed=0, extra=2):
    """rel [B][Hkv][n] -> one-layer cache with those scores."""
    rel = torch.tensor(rel, dtype=torch.float32)
    B, H, n = rel.shape
    c = random_cache(1, B, H, H, D, n + extra, n, seed=seed)
    c.rel[0, :, :, :n] = rel
    return c


def test_golden_collapsed():
    g = GOLD["collapsed"]
    c = _collapsed_cache(g["rel"])
    st, keep = oracle.collapsed_prune(c, torch.tensor([g["heads"]["budget"]] * 2, dtype=torch.int32), g["recent"], g["sink"],
                                      oracle.COLLAPSE_HEADS, max_k=8)
    assert st == oracle.OK
    assert [[i for i in row if i >= 0] for row in keep.tolist()] == g["heads"]["expect"]
    for case in g["heads_batch"]:
        c = _collapsed_cache(g["rel"])
        st, keep = oracle.collapsed_prune(c, torch.tensor([case["budget"]], dtype=torch.int32), g["recent"], g["sink"],
                                          oracle.COLLAPSE_HEADS_BATCH, max_k=8)
        assert st == oracle.OK and [i for i in keep[0].tolist() if i >= 0] == case["expect"]
        assert torch.all(c.len == case["budget"])


def test_collapsed_with_one_item_per_group_is_the_per_head_rule():
    """One KV head per sequence (and one sequence for the batch scope): the collapsed sum is the head's own score,
    so the call must leave exactly the bytes oracle_rasr_prune leaves."""
    for scope, B in ((oracle.COLLAPSE_HEADS, 3), (oracle.COLLAPSE_HEADS_BATCH, 1)):
        a = random_cache(2, B, 2, 1, 8, 300, 260, seed=3, rel_init="rand")
        a.rel[:, :, :, 50:90] = 0.5                                    # ties
        b = a.clone()
        bud = torch.tensor([[90] * B, [400] * B], dtype=torch.int32)
        st_a, keep_a = oracle.rasr_prune(a, bud, 16, 4, max_k=300)
        st_b, keep_b = oracle.collapsed_prune(b, bud.flatten() if scope == oracle.COLLAPSE_HEADS else bud[:, 0].contiguous(),
                                              16, 4, scope, max_k=300)
        assert st_a == st_b == oracle.OK and torch.equal(keep_a.reshape(keep_b.shape), keep_b)
        for name in ("k", "v", "rel", "pos", "len"):
            assert torch.equal(getattr(a, name), getattr(b, name)), name


def test_collapsed_brute_force_tiny():
    """Sum the heads with numpy fp32 in (b, h) order, enumerate every size-k superset of the protected set, and
    check that the kept set is the best one (largest collapsed sum, then lexicographically smallest), that all
    items of a group were compacted by that same list and that each kept its own rows."""
    import numpy as np
    g = torch.Generator().manual_seed(29)
    for trial in range(80):
        B = int(torch.randint(1, 3, (1,), generator=g)); H = int(torch.randint(1, 4, (1,), generator=g))
        n = int(torch.randint(3, 11, (1,), generator=g))
        sink = int(torch.randint(0, 3, (1,), generator=g)); recent = int(torch.randint(0, 3, (1,), generator=g))
        prot = set(range(min(sink, n))) | set(range(n - min(recent, n), n))
        if len(prot) >= n:
            continue
        k = int(torch.randint(len(prot), n, (1,), generator=g))
        rel = torch.randint(0, 4, (B, H, n), generator=g).float() * 0.25
        for scope in (oracle.COLLAPSE_HEADS, oracle.COLLAPSE_HEADS_BATCH):
            c = _collapsed_cache(rel.tolist(), seed=trial)
            before = c.clone()
            groups = B if scope == oracle.COLLAPSE_HEADS else 1
            st, keep = oracle.collapsed_prune(c, torch.full((groups,), k, dtype=torch.int32), recent, sink, scope, max_k=n)
            assert st == oracle.OK
            for gi in range(groups):
                members = [(gi, h) for h in range(H)] if scope == oracle.COLLAPSE_HEADS else [(b, h) for b in range(B) for h in range(H)]
                score = np.zeros(n, dtype=np.float32)
                for (b, h) in members:
                    score = (score + rel[b, h].numpy()).astype(np.float32)
                rest = [j for j in range(n) if j not in prot]
                best = min((-float(sum(score[j] for j in extra)), tuple(extra))
                           for extra in itertools.combinations(rest, k - len(prot)))
                kept = [i for i in keep[gi].tolist() if i >= 0]
                assert tuple(sorted(set(kept) - prot)) == best[1] and prot <= set(kept) and len(kept) == k
                idx = torch.tensor(kept, dtype=torch.long)
                for (b, h) in members:
                    assert int(c.len[0, b, h]) == k
                    for name in ("k", "v", "rel", "pos"):
                        assert torch.equal(getattr(c, name)[0, b, h, :k], getattr(before, name)[0, b, h, idx]), name


def test_collapsed_identical_heads_keep_what_each_head_would_keep():
    """When every head of a sequence holds the same scores the sum is a power-of-two multiple of them (4 heads):
    order and ties are unchanged, so the shared set equals every head's own set."""
    a = random_cache(1, 2, 4, 4, 8, 500, 450, seed=8, rel_init="rand")
    a.rel[:] = a.rel[:, :, :1]
    a.rel[:, :, :, 100:160] = 0.25
    b = a.clone()
    bud = torch.tensor([[120, 333]], dtype=torch.int32)
    st_a, _ = oracle.rasr_prune(a, bud, 32, 4)
    st_b, _ = oracle.collapsed_prune(b, bud.flatten(), 32, 4, oracle.COLLAPSE_HEADS)
    assert st_a == st_b == oracle.OK
    for name in ("k", "v", "rel", "pos", "len"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name


def test_collapsed_sum_is_taken_in_fp32_in_head_order():
    """Slot 1 holds (2^24, 1, 1), slot 2 holds (2^24, 2, 0).  Exactly both sum to 2^24 + 2 and the older slot 1
    would win the tie; in fp32, adding head by head, slot 1 stays at 2^24 (each +1 rounds back to even) and slot 2
    reaches 2^24 + 2, so slot 2 is the one kept.  The decision is documented as an fp32 one."""
    big = float(2 ** 24)
    rel = [[[0, big, big, 0, 0], [0, 1, 2, 0, 0], [0, 1, 0, 0, 0]]]
    c = _collapsed_cache(rel)
    st, keep = oracle.collapsed_prune(c, torch.tensor([3], dtype=torch.int32), 1, 1, oracle.COLLAPSE_HEADS, max_k=5)
    assert st == oracle.OK and [i for i in keep[0].tolist() if i >= 0] == [0, 2, 4]


def test_collapsed_special_cases():
    base = random_cache(2, 2, 4, 2, 8, 64, 50, seed=4, rel_init="rand")
    # budget >= length: identity
    c = base.clone()
    st, keep = oracle.collapsed_prune(c, torch.tensor([50, 60, 70, 80], dtype=torch.int32), 8, 2, oracle.COLLAPSE_HEADS, max_k=64)
    assert st == oracle.OK and keep[0].tolist() == list(range(50)) + [-1] * 14
    for name in ("k", "v", "rel", "pos", "len"):
        assert torch.equal(getattr(c, name), getattr(base, name))
    # heads of one sequence out of step: that group is refused and untouched, the others are pruned
    c = base.clone(); c.len[0, 1, 1] = 49
    ref = c.clone()
    st, keep = oracle.collapsed_prune(c, torch.tensor([20] * 4, dtype=torch.int32), 8, 2, oracle.COLLAPSE_HEADS, max_k=64)
    assert st == oracle.ERR_INVALID_ARG
    assert c.len[0, 1].tolist() == [50, 49] and torch.equal(c.k[0, 1], ref.k[0, 1]) and torch.all(keep[1] == -1)
    assert c.len[0, 0].tolist() == [20, 20] and c.len[1].flatten().tolist() == [20] * 4
    # protected set above the budget: exactly the protected set, flagged
    c = base.clone()
    st, keep = oracle.collapsed_prune(c, torch.tensor([5, 5], dtype=torch.int32), 8, 2, oracle.COLLAPSE_HEADS_BATCH, max_k=64)
    assert st == oracle.ERR_BUDGET and torch.all(c.len == 10)
    assert [i for i in keep[0].tolist() if i >= 0] == [0, 1] + list(range(42, 50))
    # batch scope on (B, Hkv) equals head scope on the same items seen as (1, B * Hkv)
    a = base.clone()
    b = oracle.OracleCache(2, 1, 8, 4, 8, 64, base.k.reshape(2, 1, 4, 64, 8).clone(), base.v.reshape(2, 1, 4, 64, 8).clone(),
                           base.rel.reshape(2, 1, 4, 64).clone(), base.pos.reshape(2, 1, 4, 64).clone(),
                           base.len.reshape(2, 1, 4).clone())
    bud = torch.tensor([17, 33], dtype=torch.int32)
    st_a, keep_a = oracle.collapsed_prune(a, bud, 8, 2, oracle.COLLAPSE_HEADS_BATCH, max_k=64)
    st_b, keep_b = oracle.collapsed_prune(b, bud, 8, 2, oracle.COLLAPSE_HEADS, max_k=64)
    assert st_a == st_b == oracle.OK and torch.equal(keep_a, keep_b) and torch.equal(a.k.flatten(), b.k.flatten())


# ----------------------------------------------------------------------------- quantised (e4m3) K / V storage

def _fp8_cache(L, B, Hq, Hkv, D, cap, n, seed, k_scale, v_scale):
    """Cache whose K / V bytes are random e4m3 codes (no NaN codes), with per-layer scales."""
    g = torch.Generator().manual_seed(seed)
    def codes():
        c = torch.randint(0, 256, (L, B, Hkv, cap, D), generator=g, dtype=torch.int32)
        c[(c & 0x7f) == 0x7f] = 0x30
        return c.to(torch.uint8).view(torch.float8_e4m3fn)
    rel = torch.rand((L, B, Hkv, cap), generator=g)
    pos = torch.arange(cap, dtype=torch.int32).expand(L, B, Hkv, cap).contiguous()
    return oracle.OracleCache(L, B, Hq, Hkv, D, cap, codes(), codes(), rel, pos, torch.full((L, B, Hkv), n, dtype=torch.int32),
                              k_scale=torch.tensor(k_scale, dtype=torch.float32), v_scale=torch.tensor(v_scale, dtype=torch.float32))


def test_e4m3_conversions_against_closed_forms_and_the_library():
    lib = oracle.lib()
    # decode: every code against the library's table, a few against the format's definition
    codes = torch.arange(256, dtype=torch.uint8)
    ref = codes.view(torch.float8_e4m3fn).double()
    got = torch.tensor([lib.oracle_e4m3_decode(int(c)) for c in codes], dtype=torch.float64)
    assert bool(((ref == got) | (ref.isnan() & got.isnan())).all())
    for code, value in ((0x38, 1.0), (0x7e, 448.0), (0x08, 2.0 ** -6), (0x01, 2.0 ** -9), (0x07, 7 * 2.0 ** -9), (0xb8, -1.0), (0x00, 0.0)):
        assert lib.oracle_e4m3_decode(code) == value
    # encode: exact values round-trip; midpoints between neighbours go to the even code; overflow saturates
    finite = [c for c in range(0x7f)]
    for c in finite:
        assert lib.oracle_e4m3_encode(lib.oracle_e4m3_decode(c)) == c
        assert lib.oracle_e4m3_encode(-lib.oracle_e4m3_decode(c)) == (c | 0x80)
    for c in range(0x7e):
        mid = 0.5 * (lib.oracle_e4m3_decode(c) + lib.oracle_e4m3_decode(c + 1))      # exactly representable in fp32
        assert lib.oracle_e4m3_encode(mid) == (c if c % 2 == 0 else c + 1), c
        assert lib.oracle_e4m3_encode(float(torch.nextafter(torch.tensor(mid), torch.tensor(1e9)))) == c + 1
        assert lib.oracle_e4m3_encode(float(torch.nextafter(torch.tensor(mid), torch.tensor(-1e9)))) == c
    for big in (448.0001, 464.0, 480.0, 1e6, 3e38):
        assert lib.oracle_e4m3_encode(big) == 0x7e and lib.oracle_e4m3_encode(-big) == 0xfe
    # the library's cast on random in-range values
    g = torch.Generator().manual_seed(0)
    x = (torch.randn(20000, generator=g) * torch.exp(torch.randn(20000, generator=g) * 3)).clamp(-448, 448)
    want = x.to(torch.float8_e4m3fn).view(torch.uint8)
    got = torch.tensor([lib.oracle_e4m3_encode(float(v)) for v in x.tolist()], dtype=torch.uint8)
    assert torch.equal(want, got)


def test_quantised_cache_attends_like_the_cache_of_its_dequantised_values():
    """Reading a byte x as scale * x is exact, so a quantised cache must give what the fp32 cache holding those
    products gives: the same relevance bit for bit, the same output up to the bf16 rounding of out."""
    L, B, Hq, Hkv, D, cap, n = 2, 2, 8, 2, 16, 40, 33
    ks, vs = [0.25, 0.5], [2.0, 0.125]                                  # powers of two: scale * x is exact in fp32 too
    q8 = _fp8_cache(L, B, Hq, Hkv, D, cap, n, 3, ks, vs)
    kf = q8.k.float() * torch.tensor(ks).reshape(L, 1, 1, 1, 1)
    vf = q8.v.float() * torch.tensor(vs).reshape(L, 1, 1, 1, 1)
    f32 = oracle.OracleCache(L, B, Hq, Hkv, D, cap, kf, vf, q8.rel.clone(), q8.pos.clone(), q8.len.clone())
    g = torch.Generator().manual_seed(4)
    q = (torch.randn((L, B, Hq, D), generator=g) * 0.3).to(torch.bfloat16)
    scale = torch.tensor([0.2, 0.35], dtype=torch.float32)
    st8, out8, lse8, _ = oracle.decode_attend(q8, 0, L, q, None, None, None, scale, 0.9, want_lse=True)
    st32, out32, lse32, _ = oracle.decode_attend(f32, 0, L, q.float(), None, None, None, scale, 0.9, want_lse=True)
    assert st8 == st32 == oracle.OK and out8.dtype == torch.bfloat16
    assert torch.equal(q8.rel, f32.rel) and torch.equal(lse8, lse32)
    assert (out8.float() - out32).abs().max() <= 2.0 ** -8 * out32.abs().max()
    # non-trivial scales (not powers of two) against the double-precision definition
    q8b = _fp8_cache(1, 1, 4, 1, 8, 12, 9, 5, [0.3], [1.7])
    qq = (torch.randn((1, 1, 4, 8), generator=g) * 0.5).to(torch.bfloat16)
    st, out, _, probs = oracle.decode_attend(q8b, 0, 1, qq, None, None, None, torch.tensor([0.4]), 1.0, want_probs=True)
    kd = q8b.k.double()[0, 0, 0, :9] * float(torch.tensor(0.3, dtype=torch.float32))
    vd = q8b.v.double()[0, 0, 0, :9] * float(torch.tensor(1.7, dtype=torch.float32))
    p = torch.softmax((qq.double()[0, 0] @ kd.T) * float(torch.tensor(0.4, dtype=torch.float32)), dim=-1)
    assert torch.allclose(probs[0, 0, :, :9], p, rtol=1e-12, atol=1e-15)
    assert torch.allclose(out[0, 0].double(), p @ vd, rtol=2.0 ** -8, atol=1e-6)


def test_quantised_append_rounds_like_the_library_and_saturates():
    L, B, Hq, Hkv, D, cap, n = 1, 2, 4, 2, 32, 16, 5
    ks, vs = [0.37], [3.0]
    c = _fp8_cache(L, B, Hq, Hkv, D, cap, n, 6, ks, vs)
    before = c.clone()
    g = torch.Generator().manual_seed(8)
    q = torch.randn((L, B, Hq, D), generator=g).to(torch.bfloat16)
    kn = (torch.randn((L, B, Hkv, D), generator=g) * 20).to(torch.bfloat16)
    vn = (torch.randn((L, B, Hkv, D), generator=g) * 100).to(torch.bfloat16)
    kn[0, 0, 0, :4] = torch.tensor([1e4, -1e4, 0.0, 165.76], dtype=torch.bfloat16)   # beyond 448 * 0.37: saturates
    st, *_ = oracle.decode_attend(c, 0, L, q, kn, vn, torch.tensor([7, 9], dtype=torch.int32), torch.tensor([0.1]), 0.9)
    assert st == oracle.OK and torch.all(c.len == n + 1)
    tk = kn.float() / torch.tensor(ks[0], dtype=torch.float32)
    tv = vn.float() / torch.tensor(vs[0], dtype=torch.float32)
    want_k = tk.clamp(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8)      # the library rounds, the clamp saturates
    want_v = tv.clamp(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8)
    assert torch.equal(c.k.view(torch.uint8)[0, :, :, n], want_k[0]) and torch.equal(c.v.view(torch.uint8)[0, :, :, n], want_v[0])
    assert c.k.view(torch.uint8)[0, 0, 0, n, 0] == 0x7e and c.k.view(torch.uint8)[0, 0, 0, n, 1] == 0xfe
    assert torch.equal(c.k.view(torch.uint8)[..., :n, :], before.k.view(torch.uint8)[..., :n, :])
    assert torch.equal(c.pos[0, :, :, n], torch.tensor([[7, 7], [9, 9]], dtype=torch.int32))


def test_quantised_cache_prunes_by_moving_bytes():
    c = _fp8_cache(2, 2, 4, 2, 16, 64, 50, 9, [1.0, 1.0], [1.0, 1.0])
    before = c.clone()
    st, keep = oracle.rasr_prune(c, torch.tensor([[20, 60], [33, 12]], dtype=torch.int32), 8, 2, max_k=64)
    assert st == oracle.OK
    for l in range(2):
        for b in range(2):
            for h in range(2):
                m = int(c.len[l, b, h])
                idx = keep[l, b, h, :m].long()
                assert torch.equal(c.k.view(torch.uint8)[l, b, h, :m], before.k.view(torch.uint8)[l, b, h, idx])
                assert torch.equal(c.v.view(torch.uint8)[l, b, h, :m], before.v.view(torch.uint8)[l, b, h, idx])
                assert torch.equal(c.rel[l, b, h, :m], before.rel[l, b, h, idx])
    assert c.len[0, 0].tolist() == [20, 20] and c.len[0, 1].tolist() == [50, 50]


def test_e5m2_conversions_against_closed_forms_and_the_library():
    """The second byte format: e5m2, the upper byte of an IEEE half."""
    lib = oracle.lib()
    codes = torch.arange(256, dtype=torch.uint8)
    ref = codes.view(torch.float8_e5m2).double()
    got = torch.tensor([lib.oracle_e5m2_decode(int(c)) for c in codes], dtype=torch.float64)
    assert bool(((ref == got) | (ref.isnan() & got.isnan())).all())
    for code, value in ((0x3c, 1.0), (0x7b, 57344.0), (0x04, 2.0 ** -14), (0x01, 2.0 ** -16), (0xbc, -1.0), (0x3d, 1.25)):
        assert lib.oracle_e5m2_decode(code) == value
        # a byte is the upper half of the half-precision number of the same value
        assert torch.tensor([code << 8], dtype=torch.int32).to(torch.int16).view(torch.float16).item() == value
    for c in range(0x7c):                                    # finite codes round-trip; ties go to the even code
        assert lib.oracle_e5m2_encode(lib.oracle_e5m2_decode(c)) == c
        if c < 0x7b:
            mid = 0.5 * (lib.oracle_e5m2_decode(c) + lib.oracle_e5m2_decode(c + 1))
            assert lib.oracle_e5m2_encode(mid) == (c if c % 2 == 0 else c + 1), c
            assert lib.oracle_e5m2_encode(float(torch.nextafter(torch.tensor(mid), torch.tensor(1e9)))) == c + 1
            assert lib.oracle_e5m2_encode(float(torch.nextafter(torch.tensor(mid), torch.tensor(-1e9)))) == c
    for big in (57345.0, 61440.0, 65536.0, 1e9, 3e38):     # never infinity: saturation
        assert lib.oracle_e5m2_encode(big) == 0x7b and lib.oracle_e5m2_encode(-big) == 0xfb
    g = torch.Generator().manual_seed(1)
    x = (torch.randn(20000, generator=g) * torch.exp(torch.randn(20000, generator=g) * 5)).clamp(-57344, 57344)
    want = x.to(torch.float8_e5m2).view(torch.uint8)
    got = torch.tensor([lib.oracle_e5m2_encode(float(v)) for v in x.tolist()], dtype=torch.uint8)
    assert torch.equal(want, got)


def test_e5m2_cache_attends_like_the_cache_of_its_dequantised_values():
    L, B, Hq, Hkv, D, cap, n = 1, 2, 4, 2, 16, 24, 19
    g = torch.Generator().manual_seed(14)
    def codes():
        c = torch.randint(0, 256, (L, B, Hkv, cap, D), generator=g, dtype=torch.int32)
        c[(c & 0x7c) == 0x7c] = 0x38                             # no infinities / NaNs
        c[(c & 0x7f) > 0x48] = 0x40                               # keep magnitudes moderate
        return c.to(torch.uint8).view(torch.float8_e5m2)
    k8, v8 = codes(), codes()
    rel = torch.rand((L, B, Hkv, cap), generator=g)
    pos = torch.arange(cap, dtype=torch.int32).expand(L, B, Hkv, cap).contiguous()
    ln = torch.full((L, B, Hkv), n, dtype=torch.int32)
    q8 = oracle.OracleCache(L, B, Hq, Hkv, D, cap, k8, v8, rel.clone(), pos.clone(), ln.clone(),
                            k_scale=torch.tensor([0.5]), v_scale=torch.tensor([0.25]))
    f32 = oracle.OracleCache(L, B, Hq, Hkv, D, cap, k8.float() * 0.5, v8.float() * 0.25, rel.clone(), pos.clone(), ln.clone())
    q = (torch.randn((L, B, Hq, D), generator=g) * 0.3).to(torch.bfloat16)
    kn = torch.randn((L, B, Hkv, D), generator=g).to(torch.bfloat16)
    kn[0, 0, 0, 0] = 1e9                                          # saturates at 57344 * 0.5, never infinity
    scale = torch.tensor([0.2], dtype=torch.float32)
    tp = torch.tensor([3, 4], dtype=torch.int32)
    st8, out8, _, _ = oracle.decode_attend(q8, 0, L, q, kn, kn, tp, scale, 0.9)
    # the fp32 twin appends the dequantised bytes the quantised cache stored
    kq = q8.k.float()[:, :, :, n] * 0.5
    vq = q8.v.float()[:, :, :, n] * 0.25
    st32, out32, _, _ = oracle.decode_attend(f32, 0, L, q.float(), kq.reshape(L, B, Hkv, D).contiguous(),
                                             vq.reshape(L, B, Hkv, D).contiguous(), tp, scale, 0.9)
    assert st8 == st32 == oracle.OK
    assert q8.k.view(torch.uint8)[0, 0, 0, n, 0] == 0x7b
    want = (kn.float() / 0.5).clamp(-57344, 57344).to(torch.float8_e5m2).view(torch.uint8)
    assert torch.equal(q8.k.view(torch.uint8)[0, :, :, n], want[0])
    assert torch.equal(q8.rel, f32.rel)
    assert (out8.float() - out32).abs().max() <= 2.0 ** -8 * out32.abs().max()
