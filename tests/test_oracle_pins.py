"""Pins for the CPU oracle: closed forms, invariants, textbook special cases and brute force
(Python loops, exact rationals).  None of these re-types the oracle's own formulas with the
same library calls; each is chosen so that a dropped term, a wrong sign or index, or a
transposed operand in the oracle fails it."""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import meda_oracle as O

RNG = np.random.default_rng(1234)


def _modality(n_text_head, n_vis, n_text_tail):
    return np.array([0] * n_text_head + [1] * n_vis + [0] * n_text_tail, dtype=np.uint8)


# ----------------------------------------------------------------------------- brute force

def brute_attention(q, k, q_pos, allowed):
    """P[h][i][j] with Python loops and math.exp: softmax over visible keys with allowed[j]."""
    hq, w, d = q.shape
    hkv, n, _ = k.shape
    G = hq // hkv
    P = [[[0.0] * n for _ in range(w)] for _ in range(hq)]
    for h in range(hq):
        g = h // G
        for i in range(w):
            js = [j for j in range(n) if j <= q_pos[i] and allowed[j]]
            if not js:
                continue
            logit = {j: sum(float(q[h, i, t]) * float(k[g, j, t]) for t in range(d)) / math.sqrt(d) for j in js}
            mx = max(logit.values())
            z = sum(math.exp(logit[j] - mx) for j in js)
            for j in js:
                P[h][i][j] = math.exp(logit[j] - mx) / z
    return P


def test_scores_match_bruteforce_gqa_and_causal():
    hq, hkv, w, n, d = 4, 2, 5, 13, 3
    q = RNG.normal(size=(hq, w, d))
    k = RNG.normal(size=(hkv, n, d))
    q_pos = np.arange(n - w, n)
    P = brute_attention(q, k, q_pos, [True] * n)
    want = np.zeros((hkv, n))
    for h in range(hq):
        for i in range(w):
            for j in range(n):
                want[h // (hq // hkv), j] += P[h][i][j]
    got = O.window_scores(q, k)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-14)
    # causal: the last key is seen by the last window row only
    assert got[:, n - 1].max() < (hq // hkv) * 1.0 + 1e-12
    # every softmax row sums to one: mass G * w per KV head
    np.testing.assert_allclose(got.sum(axis=1), (hq // hkv) * w, rtol=1e-12)


def test_scores_full_window_equal_column_sums_of_causal_attention():
    # window = whole prompt: Eq. 8 literally
    n, d = 9, 4
    q = RNG.normal(size=(1, n, d))
    k = RNG.normal(size=(1, n, d))
    s = np.array([[sum(q[0, i, t] * k[0, j, t] for t in range(d)) / math.sqrt(d) for j in range(n)] for i in range(n)])
    A = np.zeros((n, n))
    for i in range(n):
        e = [math.exp(s[i, j]) for j in range(i + 1)]
        for j in range(i + 1):
            A[i, j] = e[j] / sum(e)
    np.testing.assert_allclose(O.window_scores(q, k)[0], A.sum(axis=0), rtol=1e-12)


def test_entropy_uniform_is_log_nv():
    mod = _modality(3, 17, 6)
    n = mod.size
    q = np.zeros((2, 4, 8))
    k = RNG.normal(size=(2, n, 8))
    for mode in (0, 1):
        assert O.cross_modal_entropy(q, k, mod, entropy_mode=mode) == pytest.approx(math.log(17), rel=1e-13)


def test_entropy_one_hot_is_zero():
    mod = _modality(2, 10, 4)
    n, d = mod.size, 4
    k = np.zeros((1, n, d))
    k[0, 5, 0] = 80.0 * math.sqrt(d)
    q = np.zeros((1, 4, d))
    q[:, :, 0] = 1.0
    e = O.cross_modal_entropy(q, k, mod)
    assert 0.0 <= e < 1e-30


def test_entropy_two_level_closed_form():
    # m visual keys at logit a, the other visual keys at 0: H = ln Z - m a e^a / Z
    mod = _modality(4, 20, 5)
    n, d = mod.size, 4
    a, m = 1.7, 6
    k = np.zeros((1, n, d))
    vis = np.nonzero(mod == 1)[0]
    k[0, vis[:m], 1] = a * math.sqrt(d) / 2.0
    k[0, :4, 1] = 9.0    # text keys must not enter the visual softmax
    q = np.zeros((1, 3, d))
    q[:, :, 1] = 2.0
    Z = m * math.exp(a) + (20 - m)
    want = math.log(Z) - m * a * math.exp(a) / Z
    assert O.cross_modal_entropy(q, k, mod) == pytest.approx(want, rel=1e-13)


def test_entropy_head_mean_vs_mean_of_entropies():
    # two heads, each one-hot on a different visual key: mean attention has entropy ln 2,
    # the mean of the per-head entropies is 0
    mod = _modality(1, 6, 3)
    n, d = mod.size, 2
    k = np.zeros((2, n, d))
    k[0, 2, 0] = 100.0
    k[1, 4, 0] = 100.0
    q = np.zeros((2, 3, d))
    q[:, :, 0] = 10.0
    assert O.cross_modal_entropy(q, k, mod, entropy_mode=0) == pytest.approx(math.log(2), rel=1e-12)
    assert abs(O.cross_modal_entropy(q, k, mod, entropy_mode=1)) < 1e-12


def test_entropy_matches_scipy_routines():
    from scipy.special import softmax
    from scipy.stats import entropy
    mod = _modality(5, 23, 7)
    n, d, hq, hkv, w = mod.size, 8, 4, 2, 6
    q = RNG.normal(size=(hq, w, d))
    k = RNG.normal(size=(hkv, n, d))
    vis = mod == 1
    mean_attn = np.zeros((w, vis.sum()))
    per_head = 0.0
    for h in range(hq):
        logits = q[h] @ k[h // 2][vis].T / math.sqrt(d)   # window is text at the end: all visual keys visible
        p = softmax(logits, axis=1)
        mean_attn += p / hq
        per_head += entropy(p, axis=1).mean() / hq
    assert O.cross_modal_entropy(q, k, mod, entropy_mode=0) == pytest.approx(entropy(mean_attn, axis=1).mean(), rel=1e-12)
    assert O.cross_modal_entropy(q, k, mod, entropy_mode=1) == pytest.approx(per_head, rel=1e-12)


def test_entropy_bruteforce_with_visual_query_rows_and_causality():
    # interleaved layout; visual query rows in the middle see only earlier text keys
    mod = np.array([0, 0, 1, 1, 1, 0, 1, 1, 0, 0, 0], dtype=np.uint8)
    n, d, hq, hkv = mod.size, 3, 2, 1
    q_pos = np.array([8, 9, 10])
    qv_pos = np.array([2, 4, 7])
    q = RNG.normal(size=(hq, 3, d))
    qv = RNG.normal(size=(hq, 3, d))
    k = RNG.normal(size=(hkv, n, d))

    def term(qq, pos, subset):
        P = brute_attention(qq, k, pos, subset)
        rows = [i for i in range(len(pos)) if any(subset[j] for j in range(pos[i] + 1))]
        tot = 0.0
        for i in rows:
            for j in range(n):
                a = sum(P[h][i][j] for h in range(hq)) / hq
                if a > 0:
                    tot += a * math.log(a)
        return tot / len(rows)

    e_tv = term(q, q_pos, [m == 1 for m in mod])
    e_vt = term(qv, qv_pos, [m == 0 for m in mod])
    assert O.cross_modal_entropy(q, k, mod, q_pos) == pytest.approx(-e_tv, rel=1e-12)
    assert O.cross_modal_entropy(q, k, mod, q_pos, qv, qv_pos) == pytest.approx(-(e_tv + e_vt), rel=1e-12)


def test_row_stats_reproduce_the_softmax():
    mod = _modality(3, 11, 5)
    n, d, hq, hkv, w = mod.size, 4, 4, 2, 5
    q = RNG.normal(size=(hq, w, d))
    k = RNG.normal(size=(hkv, n, d))
    st = O.row_stats(q, k, mod)
    q_pos = np.arange(n - w, n)
    P = brute_attention(q, k, q_pos, [True] * n)
    PV = brute_attention(q, k, q_pos, list(mod == 1))
    for h in range(hq):
        for i in range(w):
            for j in range(n):
                if j > q_pos[i]:
                    continue
                s = float(q[h, i] @ k[h // 2, j]) / math.sqrt(d)
                assert math.exp(s - st[h, i, 0]) / st[h, i, 1] == pytest.approx(P[h][i][j], rel=1e-11)
                if mod[j] == 1:
                    assert math.exp(s - st[h, i, 2]) / st[h, i, 3] == pytest.approx(PV[h][i][j], rel=1e-11)


# ----------------------------------------------------------------------------- allocation

def test_allocation_sums_and_equal_entropies():
    b = O.allocate_budgets(np.full(5, 3.3), 103, 1000, 4)
    assert b[:, 0].tolist() == [21, 21, 21, 20, 20]
    assert b[:, 0].sum() == 103
    assert (b[:, 1] + b[:, 2] == b[:, 0]).all()
    assert b[:, 1].tolist() == [(s * 3) // 4 for s in b[:, 0]]


def test_allocation_ratio_is_exp_of_gap():
    q, state = O.bounded_quotas(O.allocation_weights(np.array([2.0, 2.0 + 1.25])), 10_000_000, 1, 10_000_000)
    assert (state == 0).all()
    assert q[1] / q[0] == pytest.approx(math.exp(1.25), rel=1e-12)
    # Eq. 7: S_l = softmax_l * (L * rho * n) when nothing is clamped
    e = RNG.uniform(3, 4, size=6)
    w = np.exp(e) / np.exp(e).sum()
    q, _ = O.bounded_quotas(O.allocation_weights(e), 6000, 1, 100000)
    np.testing.assert_allclose(q, w * 6000, rtol=1e-12)


def test_allocation_monotone_bounded_and_feasible():
    for trial in range(50):
        L = int(RNG.integers(2, 9))
        n = int(RNG.integers(50, 400))
        lo = int(RNG.integers(1, 10))
        e = RNG.uniform(0, 9, size=L)
        B = int(RNG.integers(L * lo, L * n + 1))
        b = O.allocate_budgets(e, B, n, lo)[:, 0]
        assert b.sum() == B and b.min() >= lo and b.max() <= n
        order = np.argsort(e)
        assert (np.diff(b[order]) >= 0).all()
        q, _ = O.bounded_quotas(O.allocation_weights(e), B, lo, n)
        assert q.sum() == pytest.approx(B, rel=1e-12)
        assert np.abs(b - q).max() < 1.0


def test_allocation_clamps_match_bruteforce_lambda():
    # the quotas are clip(lambda W, lo, hi) for one lambda: find it by bisection instead
    for trial in range(20):
        L = int(RNG.integers(2, 7))
        e = RNG.uniform(0, 8, size=L)
        w = O.allocation_weights(e)
        lo, hi = 3, 60
        B = int(RNG.integers(L * lo, L * hi + 1))
        a, c = 0.0, hi / w.min() * 2
        for _ in range(200):
            mid = 0.5 * (a + c)
            if np.clip(mid * w, lo, hi).sum() < B:
                a = mid
            else:
                c = mid
        want = np.clip(c * w, lo, hi)
        q, _ = O.bounded_quotas(w, B, lo, hi)
        np.testing.assert_allclose(q, want, rtol=1e-9, atol=1e-9)


def test_allocation_is_a_best_integer_vector_bruteforce():
    # among all integer vectors inside the bounds that sum to B none is closer (max deviation)
    for trial in range(12):
        L = int(RNG.integers(2, 5))
        lo, hi = 1, 9
        e = RNG.uniform(0, 3, size=L)
        B = int(RNG.integers(L * lo, L * hi + 1))
        q, _ = O.bounded_quotas(O.allocation_weights(e), B, lo, hi)
        got = O.allocate_budgets(e, B, hi, lo)[:, 0]
        best = min(max(abs(v[l] - q[l]) for l in range(L))
                   for v in itertools.product(range(lo, hi + 1), repeat=L) if sum(v) == B)
        assert max(abs(got - q)) <= best + 1e-9


def test_allocation_infeasible_and_uniform_mode():
    with pytest.raises(O.BudgetInfeasible):
        O.allocate_budgets(np.zeros(3), 2, 100, 1)
    with pytest.raises(O.BudgetInfeasible):
        O.allocate_budgets(np.zeros(3), 301, 100, 1)
    b = O.allocate_budgets(np.array([0.0, 5.0, 9.0]), 31, 100, 1, alloc_mode=1)[:, 0]
    assert b.tolist() == [11, 10, 10]


# ----------------------------------------------------------------------------- selection

def literal_eq9_eq10(a_s, mod, M, N):
    """Eq. 9 and Eq. 10 to the letter in exact rational arithmetic."""
    a = [Fraction(float(x)) for x in a_s]
    mx = max(a)
    boosted = [a[j] + mx if mod[j] == 0 else a[j] for j in range(len(a))]
    n_cand = len(a) - M
    order = sorted(range(n_cand), key=lambda j: (-boosted[j], j))
    keep = set(order[:N]) | set(range(n_cand, len(a)))
    return sorted(keep)


def test_selection_matches_literal_eq9_eq10_in_exact_arithmetic():
    for trial in range(40):
        n = int(RNG.integers(6, 30))
        mod = RNG.integers(0, 2, size=n).astype(np.uint8)
        a_s = RNG.choice([0.125, 0.25, 0.5, 1.0, 2.0], size=n) * RNG.choice([1.0, 1.0, 3.0], size=n)  # many ties
        a_s = np.maximum(a_s, 2.0 ** -10)   # strictly positive: Eq. 9's zero-score corner is excluded
        M = int(RNG.integers(0, n // 2))
        N = int(RNG.integers(0, n - M + 1))
        conserved, less = O.select_topk(a_s, mod, M, N)
        assert conserved.tolist() == literal_eq9_eq10(a_s, mod, M, N)
        assert sorted(conserved.tolist() + less.tolist()) == list(range(n))
        assert len(conserved) == M + N


def test_selection_invariants_and_text_priority():
    n = 40
    mod = _modality(5, 25, 10)
    a_s = RNG.uniform(size=n)
    conserved, less = O.select_topk(a_s, mod, 6, 9)
    assert (np.diff(conserved) > 0).all() and (np.diff(less) > 0).all()
    assert set(range(n - 6, n)) <= set(conserved.tolist())
    # 9 important among candidates [0, 34): 5 head text + 4 tail text candidates = 9 text: all chosen
    assert all(mod[j] == 0 for j in conserved)
    conserved, less = O.select_topk(a_s, mod, 6, 12)
    picked_vis = [j for j in conserved if mod[j] == 1]
    assert len(picked_vis) == 3
    vis_c = [j for j in range(n - 6) if mod[j] == 1]
    assert sorted(picked_vis) == sorted(sorted(vis_c, key=lambda j: (-a_s[j], j))[:3])


# ----------------------------------------------------------------------------- merging

def test_nearest_conserved_bruteforce_and_first_max_tiebreak():
    n, d = 17, 5
    k = RNG.normal(size=(n, d))
    k[3] = 2.5 * k[11]            # colinear twins: cosine exactly 1 up to rounding
    conserved = np.array([1, 4, 11, 12, 16])
    less = np.array([j for j in range(n) if j not in set(conserved.tolist())])
    target, u = O.nearest_conserved(k, conserved, less)
    for p, i in enumerate(less):
        best, best_s = None, None
        for s, j in enumerate(conserved):
            c = sum(k[i, t] * k[j, t] for t in range(d)) / (math.sqrt(sum(x * x for x in k[i])) * math.sqrt(sum(x * x for x in k[j])))
            assert u[p, s] == pytest.approx(c, rel=1e-12)
            if best is None or c > best:
                best, best_s = c, s
        assert target[p] == best_s
    assert target[list(less).index(3)] == 2
    # exact tie (duplicate conserved rows): the first slot wins
    k2 = np.array([[1.0, 0.0], [1.0, 0.0], [2.0, 0.0], [0.0, 1.0]])
    t2, _ = O.nearest_conserved(k2, np.array([0, 1, 3]), np.array([2]))
    assert t2.tolist() == [0]
    # zero key: similarity 0 to everything, first slot
    k3 = np.array([[0.0, 0.0], [-1.0, 0.0], [1.0, 0.0]])
    t3, u3 = O.nearest_conserved(k3, np.array([1, 2]), np.array([0]))
    assert u3.tolist() == [[0.0, 0.0]] and t3.tolist() == [0]


def test_merge_single_slot_is_arithmetic_mean_and_untouched_slots_identical():
    n, d = 12, 4
    k = RNG.normal(size=(n, d))
    v = RNG.normal(size=(n, d))
    km, vm, counts, target = O.merge_kv(k, v, np.array([7]), np.array([j for j in range(n) if j != 7]))
    np.testing.assert_allclose(km[0], k.mean(axis=0), rtol=1e-13)
    np.testing.assert_allclose(vm[0], v.mean(axis=0), rtol=1e-13)
    assert counts.tolist() == [n]
    conserved = np.array([0, 5, 9])
    less = np.array([1, 2])
    km, vm, counts, target = O.merge_kv(k, v, conserved, less)
    for s in range(3):
        if counts[s] == 1:
            assert (km[s] == k[conserved[s]]).all() and (vm[s] == v[conserved[s]]).all()


def test_merge_conserves_count_weighted_sums_and_evict_mode():
    n, d = 60, 6
    k = RNG.normal(size=(n, d))
    v = RNG.normal(size=(n, d))
    conserved = np.sort(RNG.choice(n, size=13, replace=False))
    less = np.array([j for j in range(n) if j not in set(conserved.tolist())])
    km, vm, counts, target = O.merge_kv(k, v, conserved, less)
    assert counts.sum() == n
    np.testing.assert_allclose((km * counts[:, None]).sum(axis=0), k.sum(axis=0), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose((vm * counts[:, None]).sum(axis=0), v.sum(axis=0), rtol=1e-10, atol=1e-12)
    # Eq. 12 by hand for every slot
    for s, j in enumerate(conserved):
        members = [less[p] for p in range(len(less)) if target[p] == s]
        want = (k[j] + sum((k[i] for i in members), np.zeros(d))) / (len(members) + 1)
        np.testing.assert_allclose(km[s], want, rtol=1e-12, atol=1e-14)
    ke, ve, ce, te = O.merge_kv(k, v, conserved, less, merge_mode=1)
    assert (ke == k[conserved]).all() and (ve == v[conserved]).all() and (ce == 1).all()


# ----------------------------------------------------------------------------- rounding, pass

def test_round_to_bf16_matches_torch_on_fp32_inputs():
    x = np.concatenate([RNG.normal(size=4000) * 10.0 ** RNG.integers(-6, 6, size=4000),
                        np.array([0.0, 1.0, -1.0, 1.00390625, 1.01171875, 255.5, 256.5, 3.0e38])]).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(O.round_to_bf16(x.astype(np.float64)), want)
    # a value on which fp64 -> fp32 -> bf16 would round twice: just above a bf16 tie
    y = np.array([1.00390625 + 2.0 ** -40])
    assert O.round_to_bf16(y)[0] == 1.0078125


def test_compress_pass_accounts_for_every_token():
    from paper_2502_17599_b200 import workloads as W
    wl = W.small_variant()
    layers = [tuple(t.to(torch.float64).numpy() for t in W.make_layer(wl, l)) for l in range(wl.n_layers)]
    mod = wl.modality().numpy()
    res = O.compress_pass(layers, mod, wl.global_budget, wl.min_budget, wl.dtype)
    assert res["budgets"][:, 0].sum() == wl.global_budget
    for l, per_head in enumerate(res["layers"]):
        for g, r in enumerate(per_head):
            assert len(r["conserved"]) == res["budgets"][l, 0]
            assert len(r["conserved"]) + len(r["less"]) == wl.n_tokens
            assert r["counts"].sum() == wl.n_tokens
    # a higher-entropy layer never gets a smaller budget
    order = np.argsort(res["entropy"])
    assert (np.diff(res["budgets"][order, 0]) >= 0).all()


def test_compress_pass_is_the_composition_of_its_pinned_steps():
    """The whole pass and the per-layer wrapper against the individually pinned steps called by hand,
    on a prompt whose recent and important shares differ (M != N), so that handing the two sizes over
    in the wrong order, taking the scores of another layer or head, or merging with another head's
    keys cannot pass.  The split itself is checked from its definition: the last M_l tokens are all
    kept, exactly N_l earlier ones are, and those are text tokens first, then the best-scored."""
    from paper_2502_17599_b200 import workloads as W
    wl = W.small_variant(name="pin_compose", seed=21, rho=0.3)
    n, hkv = wl.n_tokens, wl.n_kv_heads
    layers = [tuple(t.to(torch.float64).numpy() for t in W.make_layer(wl, l)) for l in range(wl.n_layers)]
    mod = wl.modality().numpy()
    res = O.compress_pass(layers, mod, wl.global_budget, wl.min_budget, wl.dtype, beta_recent=3, beta_important=1)
    ent = np.array([O.cross_modal_entropy(q, k, mod) for q, k, _ in layers])
    np.testing.assert_array_equal(res["entropy"], ent)
    budgets = O.allocate_budgets(ent, wl.global_budget, n, wl.min_budget, 3, 1)
    np.testing.assert_array_equal(res["budgets"], budgets)
    assert (budgets[:, 1] != budgets[:, 2]).all()                      # M_l != N_l: the order of the two matters
    n_text_early = [int((mod[: n - int(m)] == O.TEXT).sum()) for m in budgets[:, 1]]
    for l, (q, k, v) in enumerate(layers):
        S, M, N = (int(x) for x in budgets[l])
        a_s = O.window_scores(q, k)
        np.testing.assert_array_equal(res["scores"][l], a_s)
        for g in range(hkv):
            r = res["layers"][l][g]
            cons, less = O.select_topk(a_s[g], mod, M, N)                # (recent, important) in this order
            np.testing.assert_array_equal(r["conserved"], cons)
            np.testing.assert_array_equal(r["less"], less)
            # the split from its definition (Eq. 10), without select_topk
            kept = np.zeros(n, dtype=bool)
            kept[r["conserved"]] = True
            assert kept[n - M:].all() and int(kept[: n - M].sum()) == N
            early_text = np.nonzero((mod[: n - M] == O.TEXT))[0]
            if N >= n_text_early[l]:
                assert kept[early_text].all()                            # Eq. 9: text outranks every visual token
            else:
                assert not kept[: n - M][mod[: n - M] == O.VISUAL].any()
            # merging with this head's keys and values, and the output rounding
            km, vm, counts, target = O.merge_kv(k[g], v[g], cons, less)
            np.testing.assert_array_equal(r["target"], target)
            np.testing.assert_array_equal(r["counts"], counts)
            np.testing.assert_array_equal(r["k"], O.round_to_dtype(km, wl.dtype))
            np.testing.assert_array_equal(r["v"], O.round_to_dtype(vm, wl.dtype))
        # the per-layer wrapper alone, same arguments in the same order
        alone = O.compress_layer(k, v, a_s, mod, M, N, wl.dtype)
        for g in range(hkv):
            for key in ("conserved", "less", "target", "k", "v", "counts"):
                np.testing.assert_array_equal(alone[g][key], res["layers"][l][g][key])
    # heads of one layer and layers of one prompt really differ (a mix-up would show)
    assert not np.array_equal(res["layers"][0][0]["conserved"], res["layers"][0][1]["conserved"])
    assert not np.array_equal(res["layers"][0][0]["k"][:8], res["layers"][1][0]["k"][:8])


def test_table6_headlines_and_memory_formula():
    rows, head = [], None
    with open(os.path.join(os.path.dirname(__file__), "golden", "table6_kv_memory.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            p = line.split()
            if p[0] == "headline":
                head = (float(p[1]), float(p[2]))
            else:
                rows.append(tuple(float(x) for x in p))
    full = rows[0]
    at20 = [r for r in rows if r[0] == 20][0]
    at5 = [r for r in rows if r[0] == 5][0]
    assert round(100 * (1 - at20[2] / full[2])) == head[0]
    assert round(full[1] / at5[1], 2) == head[1]
    # the formula is linear in tokens and gives 0.5 MiB per token for the 32-layer, 32-head, d=128 fp16 model
    assert O.kv_cache_gib(1) * 1024 == 0.5
    tokens_full = full[2] / O.kv_cache_gib(1)
    assert 4900 < tokens_full < 5000


def test_decode_attention_closed_forms_and_bruteforce():
    """Eq. 3: zero query = mean of the values; a key aligned with the query and scaled up = that row's
    value; adding a constant vector to every key changes nothing; brute-force loops on a small case."""
    rng = np.random.default_rng(21)
    hq, hkv, s_rows, d = 6, 2, 37, 16
    q = rng.normal(size=(hq, d))
    k = rng.normal(size=(hkv, s_rows, d))
    v = rng.normal(size=(hkv, s_rows, d))
    np.testing.assert_allclose(O.decode_attention(np.zeros_like(q), k, v), np.repeat(v.mean(axis=1), hq // hkv, axis=0), atol=1e-12)
    k2 = k.copy()
    k2[1, 5] = 400.0 * q[4] / np.linalg.norm(q[4])           # head 4 belongs to KV group 1
    np.testing.assert_allclose(O.decode_attention(q, k2, v)[4], v[1, 5], atol=1e-9)
    np.testing.assert_allclose(O.decode_attention(q, k + rng.normal(size=(1, 1, d)), v), O.decode_attention(q, k, v), atol=1e-10)
    want = np.zeros((hq, d))
    for h in range(hq):
        g = h // (hq // hkv)
        logits = [sum(q[h][t] * k[g][j][t] for t in range(d)) / math.sqrt(d) for j in range(s_rows)]
        m = max(logits)
        w = [math.exp(x - m) for x in logits]
        z = sum(w)
        for t in range(d):
            want[h][t] = sum(w[j] * v[g][j][t] for j in range(s_rows)) / z
    np.testing.assert_allclose(O.decode_attention(q, k, v), want, atol=1e-12)



def test_blockwise_prompt_scores_helper_and_prompt_query_generator():
    """The row-block evaluation the full-size GPU test uses equals the oracle's one-shot result with the
    window equal to the prompt, and the prompt-wide query generator ends in the observation window's rows."""
    import parity as P
    from paper_2502_17599_b200 import workloads as W
    q = RNG.normal(size=(4, 37, 5))
    k = RNG.normal(size=(2, 37, 5))
    np.testing.assert_allclose(P.oracle_prompt_scores(q, k, block=8), O.window_scores(q, k), rtol=1e-12)
    wl = W.small_variant()
    q_all = W.make_prompt_queries(wl, 1)
    q_win, _, _ = W.make_layer(wl, 1)
    assert q_all.shape == (wl.n_q_heads, wl.n_tokens, wl.head_dim) and q_all.dtype == q_win.dtype
    assert torch.equal(q_all[:, -wl.window:], q_win)
    assert not torch.equal(q_all[0, :wl.window], q_all[1, :wl.window])
