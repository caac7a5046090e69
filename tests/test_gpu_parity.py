"""GPU parity: every stage of the CUDA path, called through the C ABI, against the CPU oracle on
the same seeded bits.  Stage-isolated tests feed each stage the ORACLE's upstream outputs; the
end-to-end test chains the GPU stages and re-evaluates the oracle's downstream stages on the
GPU's upstream outputs, so that one tolerated near-tie cannot cascade."""
import numpy as np
import pytest
import torch

import parity as P
from oracle import meda_oracle as O
from paper_2502_17599_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2502_17599_b200 import build
    build.build()


def _alternating_spans(n_text, n_visual, repeats, tail_text):
    """((begin, end, modality), ...): `repeats` times (text, visual), then a text tail."""
    spans, at = [], 0
    for _ in range(repeats):
        spans.append((at, at + n_text, 0)); at += n_text
        spans.append((at, at + n_visual, 1)); at += n_visual
    spans.append((at, at + tail_text, 0))
    return tuple(spans)


def small_cases():
    return [
        W.WORKLOADS["tiny"],
        W.small_variant(),                                   # bf16, GQA 3:1, ragged n = 661
        W.small_variant("small_mha_d64", n_q_heads=4, n_kv_heads=4, head_dim=64, window=17, seed=2),
        W.small_variant("small_f32_gqa", dtype="f32", n_q_heads=4, n_kv_heads=2, head_dim=128, seed=3),
        # shapes that take the tensor-core phase-A kernels (bf16, d=128, window 32 or 64)
        W.small_variant("tc_w32", window=32, seed=4),
        W.small_variant("tc_w64_wide", window=64, n_q_heads=10, n_kv_heads=2, seed=5),   # 320 query rows per KV group
        # grouped-query shapes that take the grouped scores sweep (129 .. 256 query rows per KV head, window 32):
        # 160 rows with a ragged last key block of one tile, and the full 256 rows (fewer key stages fit)
        W.small_variant("tc_w32_g5", window=32, n_q_heads=10, n_kv_heads=2, seed=6,
                        spans=((0, 37, 0), (37, 37 + 9 * 61, 1), (37 + 9 * 61, 37 + 9 * 61 + 40, 0))),   # n = 626 = 2 x 256 + 114
        W.small_variant("tc_w32_g8", window=32, n_q_heads=16, n_kv_heads=2, seed=7),
        # 224 query rows per KV head (the long-video shape) over short alternating spans: every 32-key chunk holds
        # both modalities, so the normaliser sweep takes its mixed-modality path everywhere
        W.small_variant("tc_w32_g7_alternating", window=32, n_q_heads=14, n_kv_heads=2, seed=9, frame_tokens=0,
                        spans=_alternating_spans(13, 18, 21, 40)),
        W.WORKLOADS["long_video_19k"].with_(name="long_video_19k_2l", n_layers=2),
    ]


def make_ctx(wl, **kw):
    from paper_2502_17599_b200 import binding
    return binding.Context.for_workload(wl, **kw)


@pytest.mark.parametrize("wl", small_cases(), ids=lambda w: w.name)
@pytest.mark.parametrize("entropy_mode", [0, 1])
def test_phase_a_scores_stats_entropy(wl, entropy_mode):
    ctx = make_ctx(wl, entropy_mode=entropy_mode)
    buf = P.GpuBuffers(wl)
    mod = wl.modality().numpy()
    ent2 = torch.zeros_like(buf.entropy)
    for l in range(wl.n_layers):
        (q, k, v), (qh, kh, vh) = P.layer_inputs(wl, l, "cuda")
        ctx.window_scores(l, q, k, buf.row_stats, buf.scores, buf.entropy)
        ctx.layer_entropy(l, q, k, buf.row_stats, ent2)
        ctx.check()
        P.assert_row_stats_close(P.np64(buf.row_stats), O.row_stats(qh, kh, mod))
        want_scores = O.window_scores(qh, kh)
        got_scores = P.np64(buf.scores)
        P.assert_scores_close(got_scores, want_scores)
        np.testing.assert_allclose(got_scores.sum(axis=1), (wl.n_q_heads // wl.n_kv_heads) * wl.window, rtol=1e-4)
        want_e = O.cross_modal_entropy(qh, kh, mod, entropy_mode=entropy_mode)
        P.assert_entropy_close(float(buf.entropy[l]), want_e)
        assert float(ent2[l]) == float(buf.entropy[l])      # the stand-alone sweep is the same arithmetic
        # one sweep from given normalisers: the same bits as the two-sweep call
        sc3, ent3 = torch.zeros_like(buf.scores), torch.zeros_like(buf.entropy)
        ctx.window_scores_from_stats(l, q, k, buf.row_stats, sc3, ent3)
        ctx.check()
        assert torch.equal(sc3, buf.scores) and float(ent3[l]) == float(buf.entropy[l])
    ctx.close()


def test_entropy_closed_forms_on_device():
    """Zero queries give ln(n_V); a window that sees no visual key gives 0."""
    wl = W.small_variant()
    ctx = make_ctx(wl)
    buf = P.GpuBuffers(wl)
    (q, k, v), _ = P.layer_inputs(wl, 0, "cuda")
    ctx.window_scores(0, torch.zeros_like(q), k, buf.row_stats, buf.scores, buf.entropy)
    ctx.check()
    n_vis = int((wl.modality() == 1).sum())
    assert float(buf.entropy[0]) == pytest.approx(np.log(n_vis), rel=1e-5)
    np.testing.assert_allclose(P.np64(buf.scores)[:, : wl.n_tokens - wl.window],
                               0.0 + np.sum(1.0 / (wl.n_tokens - wl.window + 1 + np.arange(wl.window))) * (wl.n_q_heads // wl.n_kv_heads),
                               rtol=1e-5)
    ctx.close()
    text_only = wl.with_(name="text_only", spans=((0, wl.n_tokens, 0),))
    ctx = make_ctx(text_only)
    ctx.window_scores(0, q, k, buf.row_stats, buf.scores, buf.entropy)
    ctx.check()
    assert float(buf.entropy[0]) == 0.0
    ctx.close()


@pytest.mark.parametrize("window", [24, 32, 64])
@pytest.mark.parametrize("modality", [0, 1])
def test_single_modality_prompts_on_both_phase_a_paths(window, modality):
    """A prompt of text alone has no cross-modal attention (entropy 0); a prompt of visual tokens alone has
    text-to-vision attention equal to the whole attention.  Windows 32 and 64 take the tensor-core kernels,
    24 the CUDA-core ones; scores, normalisers and entropy against the oracle, then a selection."""
    base = W.small_variant(window=window, seed=12)
    wl = base.with_(name=f"one_modality_{modality}", spans=((0, base.n_tokens, modality),), frame_tokens=0)
    mod = wl.modality().numpy()
    ctx = make_ctx(wl)
    buf = P.GpuBuffers(wl)
    (q, k, v), (qh, kh, vh) = P.layer_inputs(wl, 0, "cuda")
    ctx.window_scores(0, q, k, buf.row_stats, buf.scores, buf.entropy)
    ctx.check()
    P.assert_row_stats_close(P.np64(buf.row_stats), O.row_stats(qh, kh, mod))
    a_s = O.window_scores(qh, kh)
    P.assert_scores_close(P.np64(buf.scores), a_s)
    want_e = O.cross_modal_entropy(qh, kh, mod)
    if modality == 0:
        assert want_e == 0.0 and float(buf.entropy[0]) == 0.0
    else:
        assert want_e > 0.0
        P.assert_entropy_close(float(buf.entropy[0]), want_e)
    S = wl.n_tokens // 3
    M = (3 * S) // 4
    budgets = torch.tensor([[S, M, S - M]] * wl.n_layers, dtype=torch.int32, device="cuda")
    ctx.select_topk(0, buf.scores, budgets, buf.idx_c, buf.idx_less, buf.cap)
    ctx.check()
    got = P.np64(buf.scores)
    for g in range(wl.n_kv_heads):
        P.compare_selection(buf.idx_c[g, :S].cpu().numpy(), got[g], mod, M, S - M)
    ctx.close()


@pytest.mark.parametrize("alloc_mode", [0, 1])
def test_allocate_budgets_bit_exact(alloc_mode):
    rng = np.random.default_rng(7)
    for trial in range(30):
        L = int(rng.integers(1, 40))
        n = int(rng.integers(64, 5000))
        lo = int(rng.integers(1, 64))
        B = int(rng.integers(L * lo, L * n + 1))
        if trial == 0:
            B = L * lo
        if trial == 1:
            B = L * n
        wl = W.small_variant().with_(n_layers=L)
        ctx = make_ctx(wl, n_layers=L, n_tokens=n, spans=((0, n, 1),), window=min(24, n), global_budget=B,
                       min_budget=lo, alloc_mode=alloc_mode)
        ent = rng.uniform(0.0, np.log(n), size=L).astype(np.float32)
        if trial % 5 == 2:
            ent[:] = ent[0]
        e_dev = torch.from_numpy(ent).cuda()
        budgets = torch.zeros((L, 3), dtype=torch.int32, device="cuda")
        ctx.allocate_budgets(e_dev, budgets)
        ctx.check()
        want = O.allocate_budgets(ent.astype(np.float64), B, n, lo, alloc_mode=alloc_mode)
        np.testing.assert_array_equal(budgets.cpu().numpy(), want)
        assert int(budgets[:, 0].sum()) == B
        ctx.close()


@pytest.mark.parametrize("wl", small_cases(), ids=lambda w: w.name)
def test_select_topk_against_oracle_scores(wl):
    ctx = make_ctx(wl)
    buf = P.GpuBuffers(wl)
    mod = wl.modality().numpy()
    n = wl.n_tokens
    rng = np.random.default_rng(11)
    (q, k, v), (qh, kh, vh) = P.layer_inputs(wl, 0, "cuda")
    a_s = O.window_scores(qh, kh).astype(np.float32)
    a_s[:, 5:9] = a_s[:, 5:6]          # exact ties: lowest index must win
    scores = torch.from_numpy(a_s).cuda()
    cases = [(n // 4, n // 8), (0, 5), (7, 0), (n, 0), (n // 2, n - n // 2), (3, int((mod[: n - 3] == 0).sum())), (1, 1)]
    swaps = 0
    for M, N in cases:
        budgets = torch.tensor([[M + N, M, N]] * wl.n_layers, dtype=torch.int32, device="cuda")
        buf.idx_c.fill_(-1)
        buf.idx_less.fill_(-1)
        ctx.select_topk(0, scores, budgets, buf.idx_c, buf.idx_less, buf.cap)
        ctx.check()
        for g in range(wl.n_kv_heads):
            cons = buf.idx_c[g, : M + N].cpu().numpy()
            less = buf.idx_less[g, : n - M - N].cpu().numpy()
            swaps += P.compare_selection(cons, a_s[g].astype(np.float64), mod, M, N)
            assert (np.diff(less) > 0).all()
            assert sorted(cons.tolist() + less.tolist()) == list(range(n))
            assert (buf.idx_c[g, M + N:] == -1).all() and (buf.idx_less[g, n - M - N:] == -1).all()
    assert swaps == 0      # identical fp32 scores on both sides: no tolerance needed
    ctx.close()


def test_select_reports_capacity_and_bad_budget_rows():
    from paper_2502_17599_b200 import binding as B
    wl = W.small_variant()
    ctx = make_ctx(wl)
    buf = P.GpuBuffers(wl, cap=64)
    scores = torch.rand((wl.n_kv_heads, wl.n_tokens), device="cuda")
    budgets = torch.tensor([[100, 75, 25]] * wl.n_layers, dtype=torch.int32, device="cuda")
    ctx.select_topk(0, scores, budgets, buf.idx_c, buf.idx_less, 64)
    assert ctx.poll_status() == B.MEDA_ERR_WORKSPACE
    assert (buf.idx_c == -1).all()
    assert ctx.poll_status() == B.MEDA_OK           # cleared by the poll
    bad = torch.tensor([[10, 8, 3]] * wl.n_layers, dtype=torch.int32, device="cuda")
    ctx.select_topk(0, scores, bad, buf.idx_c, buf.idx_less, 64)
    assert ctx.poll_status() == B.MEDA_ERR_BUDGET_INFEASIBLE
    with pytest.raises(B.MedaError):
        ctx.select_topk(wl.n_layers, scores, budgets, buf.idx_c, buf.idx_less, 64)
    ctx.close()


@pytest.mark.parametrize("wl", small_cases(), ids=lambda w: w.name)
@pytest.mark.parametrize("merge_mode", [0, 1])
def test_merge_kv_against_oracle_sets(wl, merge_mode, parity_report):
    ctx = make_ctx(wl, merge_mode=merge_mode)
    buf = P.GpuBuffers(wl)
    mod = wl.modality().numpy()
    n = wl.n_tokens
    near_ties = 0
    for l, (M, N) in enumerate([(n // 8, n // 16), (wl.window * 3 // 4, wl.window - wl.window * 3 // 4)][: wl.n_layers]):
        (q, k, v), (qh, kh, vh) = P.layer_inputs(wl, l, "cuda")
        a_s = O.window_scores(qh, kh)
        S = M + N
        sets = [O.select_topk(a_s[g], mod, M, N) for g in range(wl.n_kv_heads)]
        for g, (c, ls) in enumerate(sets):
            buf.idx_c[g, :S] = torch.from_numpy(c.astype(np.int32)).cuda()
            buf.idx_less[g, : n - S] = torch.from_numpy(ls.astype(np.int32)).cuda()
        budgets = torch.tensor([[S, M, N]] * wl.n_layers, dtype=torch.int32, device="cuda")
        buf.k_out.fill_(7.0)
        ctx.merge_kv(l, k, v, budgets, buf.idx_c, buf.idx_less, buf.k_out, buf.v_out, buf.counts, buf.target, buf.cap)
        ctx.check()
        for g, (c, ls) in enumerate(sets):
            tgt = buf.target[g, : n - S].cpu().numpy() if merge_mode == 0 else np.zeros(0, dtype=np.int64)
            if merge_mode == 0:
                near_ties += P.compare_targets(tgt, kh[g], c, ls)
            P.compare_merged(P.np64(buf.k_out[g, :S]), P.np64(buf.v_out[g, :S]), buf.counts[g, :S].cpu().numpy(),
                             kh[g], vh[g], c, ls, tgt, wl.dtype, merge_mode)
            assert (buf.k_out[g, S:] == 7.0).all()       # rows past S_l are left untouched
    parity_report(f"merge_kv on the oracle's sets, {wl.name}, merge_mode {merge_mode}: tolerated arg-max near-ties {near_ties}")
    ctx.close()


@pytest.mark.parametrize("S", [96, 97, 384, 385, 512, 513, 1024])
def test_merge_at_the_budgets_where_the_kernels_switch(S):
    """The layer's slot count decides on the device which arg-max kernel works (streaming up to 384 slots,
    row-gathering above) and how many passes the grouping sort executes (one up to 512 slots): both sides of
    each switch, and of a slot-tile border, on a prompt of 2,857 tokens, against the oracle."""
    wl = W.small_variant("switch_2857", spans=W._spans((37, 0), (45 * 61, 1), (75, 0)), window=32, seed=13)
    n = wl.n_tokens
    ctx = make_ctx(wl)
    buf = P.GpuBuffers(wl)
    mod = wl.modality().numpy()
    (q, k, v), (qh, kh, vh) = P.layer_inputs(wl, 0, "cuda")
    a_s = O.window_scores(qh, kh)
    M = (3 * S) // 4
    N = S - M
    sets = [O.select_topk(a_s[g], mod, M, N) for g in range(wl.n_kv_heads)]
    for g, (c, ls) in enumerate(sets):
        buf.idx_c[g, :S] = torch.from_numpy(c.astype(np.int32)).cuda()
        buf.idx_less[g, : n - S] = torch.from_numpy(ls.astype(np.int32)).cuda()
    budgets = torch.tensor([[S, M, N]] * wl.n_layers, dtype=torch.int32, device="cuda")
    buf.k_out.fill_(7.0)
    buf.target.fill_(-1)
    ctx.merge_kv(0, k, v, budgets, buf.idx_c, buf.idx_less, buf.k_out, buf.v_out, buf.counts, buf.target, buf.cap)
    ctx.check()
    for g, (c, ls) in enumerate(sets):
        tgt = buf.target[g, : n - S].cpu().numpy()
        assert (buf.target[g, n - S:] == -1).all()       # nothing written past the less-important list
        P.compare_targets(tgt, kh[g], c, ls)
        P.compare_merged(P.np64(buf.k_out[g, :S]), P.np64(buf.v_out[g, :S]), buf.counts[g, :S].cpu().numpy(),
                         kh[g], vh[g], c, ls, tgt, wl.dtype)
        assert int(buf.counts[g, :S].sum()) == n
        assert (buf.k_out[g, S:] == 7.0).all()
    ctx.close()


def test_merge_special_cases_on_device():
    """Duplicate keys merge into their twin; a single conserved slot becomes the arithmetic mean."""
    wl = W.small_variant("special", n_layers=1, frame_rho=0.0, salient_frac=0.0)
    ctx = make_ctx(wl)
    buf = P.GpuBuffers(wl)
    n = wl.n_tokens
    (q, k, v), _ = P.layer_inputs(wl, 0, "cuda")
    k = k.clone()
    k[:, 10] = k[:, 600] * 2           # colinear twin of conserved row 600 (exact in bf16)
    kh, vh = P.np64(k), P.np64(v)
    cons = np.array([3, 200, 600, 660])
    less = np.setdiff1d(np.arange(n), cons)
    for g in range(wl.n_kv_heads):
        buf.idx_c[g, :4] = torch.from_numpy(cons.astype(np.int32)).cuda()
        buf.idx_less[g, : n - 4] = torch.from_numpy(less.astype(np.int32)).cuda()
    budgets = torch.tensor([[4, 3, 1]], dtype=torch.int32, device="cuda")
    ctx.merge_kv(0, k, v, budgets, buf.idx_c, buf.idx_less, buf.k_out, buf.v_out, buf.counts, buf.target, buf.cap)
    ctx.check()
    assert (buf.target[:, list(less).index(10)] == 2).all()
    # one slot: mean of all rows
    for g in range(wl.n_kv_heads):
        buf.idx_c[g, :1] = 0
        buf.idx_less[g, : n - 1] = torch.arange(1, n, dtype=torch.int32, device="cuda")
    budgets = torch.tensor([[1, 1, 0]], dtype=torch.int32, device="cuda")
    ctx.merge_kv(0, k, v, budgets, buf.idx_c, buf.idx_less, buf.k_out, buf.v_out, buf.counts, buf.target, buf.cap)
    ctx.check()
    assert (buf.counts[:, 0] == n).all()
    np.testing.assert_allclose(P.np64(buf.k_out[:, 0]), kh.mean(axis=1), atol=2e-2)
    np.testing.assert_allclose(P.np64(buf.v_out[:, 0]), vh.mean(axis=1), atol=2e-2)
    ctx.close()


def reseeded_cases():
    """The first three benchmark configurations under two more seeds (two layers each of the larger ones)."""
    out = []
    for seed in (1, 2):
        out.append(W.WORKLOADS["tiny"].with_(name=f"tiny_seed{seed}", seed=seed))
        out.append(W.WORKLOADS["multi_image_8k"].with_(name=f"multi_image_8k_2l_seed{seed}", n_layers=2, seed=seed))
        out.append(W.WORKLOADS["long_video_19k"].with_(name=f"long_video_19k_2l_seed{seed}", n_layers=2, seed=seed))
    return out


@pytest.mark.parametrize("wl", small_cases() + reseeded_cases(), ids=lambda w: w.name)
def test_end_to_end_with_teacher_forcing(wl, parity_report):
    ctx = make_ctx(wl)
    buf = P.GpuBuffers(wl)
    mod = wl.modality().numpy()
    n = wl.n_tokens
    dev, host, scores = [], [], []
    for l in range(wl.n_layers):
        d_, h_ = P.layer_inputs(wl, l, "cuda")
        dev.append(d_)
        host.append(h_)
        sc = torch.zeros_like(buf.scores)
        ctx.window_scores(l, d_[0], d_[1], buf.row_stats, sc, buf.entropy)
        scores.append(sc)
    ctx.allocate_budgets(buf.entropy, buf.budgets)
    ctx.check()
    ent = P.np64(buf.entropy)
    for l in range(wl.n_layers):
        P.assert_entropy_close(ent[l], O.cross_modal_entropy(host[l][0], host[l][1], mod))
    budgets = buf.budgets.cpu().numpy()
    np.testing.assert_array_equal(budgets, O.allocate_budgets(ent, wl.global_budget, n, wl.min_budget))
    raw = O.allocate_budgets(np.array([O.cross_modal_entropy(h[0], h[1], mod) for h in host]), wl.global_budget, n, wl.min_budget)
    unforced = int((raw != budgets).any(axis=1).sum())
    swaps = ties = 0
    buf2 = P.GpuBuffers(wl)
    for l in range(wl.n_layers):
        S, M, N = (int(x) for x in budgets[l])
        ctx.select_topk(l, scores[l], buf.budgets, buf.idx_c, buf.idx_less, buf.cap)
        ctx.merge_kv(l, dev[l][1], dev[l][2], buf.budgets, buf.idx_c, buf.idx_less, buf.k_out, buf.v_out,
                     buf.counts, buf.target, buf.cap)
        ctx.compress_layer(l, dev[l][1], dev[l][2], scores[l], buf.budgets, buf2.k_out, buf2.v_out, buf2.counts,
                           buf2.idx_c, buf2.cap)
        ctx.check()
        a_gpu = P.np64(scores[l])
        a_or = O.window_scores(host[l][0], host[l][1])
        P.assert_scores_close(a_gpu, a_or)
        # the fused entry point is the same arithmetic as select + merge
        assert torch.equal(buf.idx_c[:, :S], buf2.idx_c[:, :S]) and torch.equal(buf.counts[:, :S], buf2.counts[:, :S])
        assert torch.equal(buf.k_out[:, :S], buf2.k_out[:, :S]) and torch.equal(buf.v_out[:, :S], buf2.v_out[:, :S])
        for g in range(wl.n_kv_heads):
            cons = buf.idx_c[g, :S].cpu().numpy().astype(np.int64)
            less = buf.idx_less[g, : n - S].cpu().numpy().astype(np.int64)
            # selection is compared on the ORACLE's scores with the swap tolerance
            swaps += P.compare_selection(cons, a_or[g], mod, M, N)
            np.testing.assert_array_equal(less, np.setdiff1d(np.arange(n), cons))
            tgt = buf.target[g, : n - S].cpu().numpy()
            ties += P.compare_targets(tgt, host[l][1][g], cons, less)
            P.compare_merged(P.np64(buf.k_out[g, :S]), P.np64(buf.v_out[g, :S]), buf.counts[g, :S].cpu().numpy(),
                             host[l][1][g], host[l][2][g], cons, less, tgt, wl.dtype)
    parity_report(f"end to end, {wl.name}: budget rows differing from the un-forced oracle {unforced} of {wl.n_layers}, "
                  f"tolerated selection swaps {swaps}, tolerated arg-max near-ties {ties}")
    ctx.close()


def test_contexts_of_different_shapes_coexist():
    """A context created later with a smaller shape must not shrink what an earlier one may launch."""
    big = W.small_variant("coexist_big", dtype="f32", n_q_heads=2, n_kv_heads=2, window=96, seed=6)
    small = W.small_variant("coexist_small", dtype="f32", n_q_heads=2, n_kv_heads=2, window=8, seed=6)
    ctx_big = make_ctx(big)
    ctx_small = make_ctx(small)
    buf = P.GpuBuffers(big)
    (q, k, v), (qh, kh, vh) = P.layer_inputs(big, 0, "cuda")
    ctx_big.window_scores(0, q, k, buf.row_stats, buf.scores, buf.entropy)
    ctx_big.check()
    P.assert_scores_close(P.np64(buf.scores), O.window_scores(qh, kh))
    ctx_small.close()
    ctx_big.close()


def test_select_beyond_cluster_capacity_uses_the_single_block_kernel():
    """A head whose keys do not fit one cluster's shared memory (n > 393,216) is selected by the
    single-block kernel; same ranking and tie-break."""
    n = 400_003
    wl = W.small_variant("select_400k", dtype="f32", n_layers=1, n_q_heads=1, n_kv_heads=1, head_dim=64, window=8,
                         spans=((0, 1000, 0), (1000, n - 500, 1), (n - 500, n, 0)), rho=0.1, frame_tokens=0)
    ctx = make_ctx(wl)
    rng = np.random.default_rng(5)
    a_s = rng.random(n).astype(np.float32)
    a_s[1234:1300] = a_s[1234]                      # a run of exact ties
    mod = wl.modality().numpy()
    scores = torch.from_numpy(a_s[None]).cuda()
    idx_c = torch.full((1, n), -1, dtype=torch.int32, device="cuda")
    idx_l = torch.full((1, n), -1, dtype=torch.int32, device="cuda")
    for M, N in ((3000, 1040), (10, 2000)):
        budgets = torch.tensor([[M + N, M, N]], dtype=torch.int32, device="cuda")
        ctx.select_topk(0, scores, budgets, idx_c, idx_l, n)
        ctx.check()
        assert P.compare_selection(idx_c[0, : M + N].cpu().numpy(), a_s.astype(np.float64), mod, M, N) == 0
        less = idx_l[0, : n - M - N].cpu().numpy()
        assert (np.diff(less) > 0).all() and less.size + M + N == n
    ctx.close()


@pytest.mark.parametrize("n", [150_001, 300_017])
def test_select_with_several_compaction_rounds_per_block(n):
    """Between 131,072 and 393,216 tokens a block of the selection cluster owns more tokens than one compaction
    round takes (16 per thread): two rounds at 150K, three at 300K, the last one ragged.  Same ranking and
    tie-break as everywhere, with a run of exact ties that straddles a round's border."""
    wl = W.small_variant(f"select_{n}", dtype="f32", n_layers=1, n_q_heads=1, n_kv_heads=1, head_dim=64, window=8,
                         spans=((0, 1000, 0), (1000, n - 500, 1), (n - 500, n, 0)), rho=0.1, frame_tokens=0)
    ctx = make_ctx(wl)
    rng = np.random.default_rng(6)
    a_s = rng.random(n).astype(np.float32)
    a_s[16_300:16_500] = a_s[16_300]                # exact ties across the first round's border of block 0
    mod = wl.modality().numpy()
    scores = torch.from_numpy(a_s[None]).cuda()
    idx_c = torch.full((1, n), -1, dtype=torch.int32, device="cuda")
    idx_l = torch.full((1, n), -1, dtype=torch.int32, device="cuda")
    # third budget: every text candidate, every visual candidate above the tied score and 100 of the 200 tied ones
    # (the lowest indices), so that the threshold falls inside the run of ties
    above = int((a_s[1000: n - 3000] > a_s[16_300]).sum())
    for M, N in ((3000, 1040), (10, 2000), (3000, 1000 + above + 100)):
        budgets = torch.tensor([[M + N, M, N]], dtype=torch.int32, device="cuda")
        ctx.select_topk(0, scores, budgets, idx_c, idx_l, n)
        ctx.check()
        assert P.compare_selection(idx_c[0, : M + N].cpu().numpy(), a_s.astype(np.float64), mod, M, N) == 0
        less = idx_l[0, : n - M - N].cpu().numpy()
        assert (np.diff(less) > 0).all() and less.size + M + N == n
        assert np.intersect1d(less, idx_c[0, : M + N].cpu().numpy()).size == 0
    ctx.close()


@pytest.mark.parametrize("wl", [
    W.small_variant(),                                                          # CUDA-core kernels for both terms
    W.small_variant("evt_tc_w32", window=32, seed=4),                           # E_TV on the tensor cores, E_VT on CUDA cores
    W.small_variant("evt_f32", dtype="f32", n_q_heads=4, n_kv_heads=2, head_dim=64, seed=3),
    # the prompt opens with an image: its first visual rows see no text key and drop out of the mean
    W.small_variant("evt_visual_first", spans=((0, 200, 1), (200, 260, 0), (260, 600, 1), (600, 661, 0)), frame_tokens=0, seed=8),
], ids=lambda w: w.name)
@pytest.mark.parametrize("entropy_mode", [0, 1])
def test_cross_modal_entropy_with_the_vision_to_text_term(wl, entropy_mode):
    """E_CM = -(E_TV + E_VT) of Eq. 5-6 with a window of visual query rows, in one call and in two."""
    ctx = make_ctx(wl, entropy_mode=entropy_mode)
    buf = P.GpuBuffers(wl)
    mod = wl.modality().numpy()
    n_rows = 19
    for l in range(2):
        (q, k, v), (qh, kh, vh) = P.layer_inputs(wl, l, "cuda")
        qv, pos = W.make_visual_queries(wl, l, n_rows, "cuda")
        want = O.cross_modal_entropy(qh, kh, mod, q_vis=P.np64(qv), q_vis_pos=pos.cpu().numpy().astype(np.int64),
                                     entropy_mode=entropy_mode)
        want_tv = O.cross_modal_entropy(qh, kh, mod, entropy_mode=entropy_mode)
        assert abs(want - want_tv) > 1e-3                     # the extra term is really there
        ctx.window_scores(l, q, k, buf.row_stats, buf.scores, buf.entropy)        # writes -E_TV
        both = torch.zeros_like(buf.entropy)
        ctx.layer_entropy(l, q, k, buf.row_stats, both, q_vis=qv, q_vis_pos=pos, n_vis_rows=n_rows)
        ctx.layer_entropy(l, None, k, None, buf.entropy, q_vis=qv, q_vis_pos=pos, n_vis_rows=n_rows)   # adds -E_VT
        ctx.check()
        P.assert_entropy_close(float(both[l]), want)
        assert float(buf.entropy[l]) == float(both[l])
    ctx.close()



@pytest.mark.parametrize("wl", small_cases(), ids=lambda w: w.name)
def test_decode_attention_over_compressed_and_full_caches(wl):
    """Eq. 3 on the device: one new token's queries over the compacted cache of a layer (row count read
    from the budgets on the device) and over the full cache (row count given)."""
    group = wl.n_q_heads // wl.n_kv_heads
    if group not in (1, 2, 3, 4, 7, 8) or wl.head_dim not in (64, 128):
        pytest.skip("shape outside the decoding kernel's list")
    ctx = make_ctx(wl)
    buf = P.GpuBuffers(wl)
    n = wl.n_tokens
    (q, k, v), (qh, kh, vh) = P.layer_inputs(wl, 0, "cuda")
    ctx.window_scores(0, q, k, buf.row_stats, buf.scores, buf.entropy)
    S = max(wl.window, n // 5)
    M = (3 * S) // 4
    budgets = torch.tensor([[S, M, S - M]] * wl.n_layers, dtype=torch.int32, device="cuda")
    ctx.compress_layer(0, k, v, buf.scores, budgets, buf.k_out, buf.v_out, buf.counts, buf.idx_c, buf.cap)
    q_new = q[:, -1, :].contiguous()                       # the last window row stands in for the new token's query
    out = torch.zeros((wl.n_q_heads, wl.head_dim), dtype=torch.float32, device="cuda")
    ctx.decode_attention(0, q_new, buf.k_out, buf.v_out, out, budgets=budgets)
    ctx.check()
    want = O.decode_attention(P.np64(q_new), P.np64(buf.k_out[:, :S]), P.np64(buf.v_out[:, :S]))
    np.testing.assert_allclose(P.np64(out), want, rtol=1e-4, atol=1e-4)
    ctx.decode_attention(0, q_new, k, v, out, n_rows=n)
    ctx.check()
    np.testing.assert_allclose(P.np64(out), O.decode_attention(P.np64(q_new), kh, vh), rtol=1e-4, atol=1e-4)
    ctx.close()


def test_degenerate_sizes_on_the_tensor_core_paths():
    """A prompt shorter than one tile (n = 97 < 128 keys, one ragged tile everywhere), and budgets at both
    ends: every token conserved (nothing to merge: outputs are the inputs) and the smallest budget."""
    n = 97
    wl = W.small_variant("short_prompt", spans=((0, 11, 0), (11, 70, 1), (70, 97, 0)), window=32, frame_tokens=0,
                         salient_frac=0.0, rho=0.4, seed=9)
    assert wl.n_tokens == n
    ctx = make_ctx(wl)
    buf = P.GpuBuffers(wl)
    mod = wl.modality().numpy()
    (q, k, v), (qh, kh, vh) = P.layer_inputs(wl, 0, "cuda")
    ctx.window_scores(0, q, k, buf.row_stats, buf.scores, buf.entropy)
    ctx.check()
    P.assert_scores_close(P.np64(buf.scores), O.window_scores(qh, kh))
    P.assert_entropy_close(float(buf.entropy[0]), O.cross_modal_entropy(qh, kh, mod))
    a_s = P.np64(buf.scores)
    for S in (n, wl.window, 1):
        M = (3 * S) // 4
        budgets = torch.tensor([[S, M, S - M]] * wl.n_layers, dtype=torch.int32, device="cuda")
        buf.k_out.fill_(7.0)
        ctx.select_topk(0, buf.scores, budgets, buf.idx_c, buf.idx_less, buf.cap)
        ctx.merge_kv(0, k, v, budgets, buf.idx_c, buf.idx_less, buf.k_out, buf.v_out, buf.counts, buf.target, buf.cap)
        ctx.check()
        for g in range(wl.n_kv_heads):
            cons = buf.idx_c[g, :S].cpu().numpy().astype(np.int64)
            less = buf.idx_less[g, : n - S].cpu().numpy().astype(np.int64)
            assert P.compare_selection(cons, a_s[g], mod, M, S - M) == 0
            tgt = buf.target[g, : n - S].cpu().numpy()
            P.compare_targets(tgt, kh[g], cons, less)
            P.compare_merged(P.np64(buf.k_out[g, :S]), P.np64(buf.v_out[g, :S]), buf.counts[g, :S].cpu().numpy(),
                             kh[g], vh[g], cons, less, tgt, wl.dtype)
            assert int(buf.counts[g, :S].sum()) == n
        if S == n:
            assert torch.equal(buf.k_out[:, :n], k) and torch.equal(buf.v_out[:, :n], v) and (buf.counts[:, :n] == 1).all()
        assert (buf.k_out[:, S:] == 7.0).all()
    ctx.close()


@pytest.mark.parametrize("wl", [W.small_variant("host_path_tc", window=32, seed=14), W.WORKLOADS["tiny"]],
                         ids=lambda w: w.name)
def test_pass_from_pinned_host_buffers_returns_what_the_device_pass_holds(wl):
    """The host-buffer variant of the whole pass (inputs copied in layer by layer while earlier layers are
    processed, results copied out layer by layer while later layers are compressed) gives the same bits as
    the pass over device-resident inputs, and reports the bytes it moved."""
    from paper_2502_17599_b200.pipeline import CompressionPass
    L = wl.n_layers
    qs, ks, vs = [], [], []
    for l in range(L):
        q, k, v = W.make_layer(wl, l, "cuda")
        qs.append(q); ks.append(k); vs.append(v)
    cp = CompressionPass(wl)
    cp.run(qs, ks, vs)
    cp.check()
    budgets = cp.budgets.cpu()
    want = {name: [src[l][:, : int(budgets[l, 0])].cpu() for l in range(L)]
            for name, src in (("k", cp.k_out), ("v", cp.v_out), ("counts", cp.counts), ("idx", cp.idx_c))}
    q_h = [t.cpu().pin_memory() for t in qs]
    k_h = [t.cpu().pin_memory() for t in ks]
    v_h = [t.cpu().pin_memory() for t in vs]
    staging = {"q": [torch.zeros_like(t) for t in qs], "k": [torch.zeros_like(t) for t in ks],
               "v": [torch.zeros_like(t) for t in vs]}
    out_host = cp.alloc_host_outputs()
    for _ in range(2):
        for name in ("k", "v", "counts", "idx"):
            for t in out_host[name]:
                t.zero_()
        h2d, d2h = cp.run_from_host(q_h, k_h, v_h, staging, out_host)
        cp.check()
        assert torch.equal(out_host["budgets"], budgets)
        for name in ("k", "v", "counts", "idx"):
            for l in range(L):
                assert torch.equal(out_host[name][l], want[name][l]), (name, l)
        assert h2d == sum(t.numel() * t.element_size() for t in q_h + k_h + v_h)
        assert d2h == budgets.numel() * 4 + sum(t.numel() * t.element_size()
                                                for name in ("k", "v", "counts", "idx") for t in out_host[name])
    cp.close()


@pytest.mark.parametrize("wl", [
    W.small_variant("capacity_2857", spans=W._spans((37, 0), (45 * 61, 1), (75, 0)), window=32, n_layers=6,
                    rho=0.25, seed=15),
    W.small_variant("capacity_f32", dtype="f32", n_q_heads=4, n_kv_heads=2, head_dim=128, n_layers=3, seed=16),
], ids=lambda w: w.name)
def test_output_capacity_smaller_than_the_prompt_gives_the_same_rows(wl):
    """Outputs sized for the largest layer budget instead of the whole prompt (the stride of the kept-index
    list and of the compacted caches changes in every phase-B kernel) hold the same bits in their live rows."""
    from paper_2502_17599_b200.pipeline import CompressionPass
    L, n = wl.n_layers, wl.n_tokens
    qs, ks, vs = [], [], []
    for l in range(L):
        q, k, v = W.make_layer(wl, l, "cuda")
        qs.append(q); ks.append(k); vs.append(v)
    full = CompressionPass(wl)
    full.run(qs, ks, vs)
    full.check()
    budgets = full.budgets.cpu().numpy()
    s_max = int(budgets[:, 0].max())
    assert s_max < n
    assert budgets[:, 0].min() <= 384 or wl.dtype != "bf16"      # both arg-max kernels take part
    tight = CompressionPass(wl, row_capacity=s_max)
    tight.run(qs, ks, vs)
    tight.check()
    assert torch.equal(tight.budgets, full.budgets)
    for l in range(L):
        S = int(budgets[l, 0])
        for a, b in ((tight.k_out, full.k_out), (tight.v_out, full.v_out), (tight.counts, full.counts),
                     (tight.idx_c, full.idx_c)):
            assert torch.equal(a[l][:, :S], b[l][:, :S]), l
    # one row too few for the largest layer is reported, not written past
    short = CompressionPass(wl, row_capacity=s_max - 1)
    short.run(qs, ks, vs)
    with pytest.raises(Exception):
        short.check()
    for c in (full, tight, short):
        c.close()
