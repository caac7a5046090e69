"""GPU parity at the full benchmark sizes, in the launch configuration bench.py times (the
CompressionPass sequence: window_scores per layer, allocate_budgets, compress_layer per layer).

Phase A costs the oracle a window-by-prompt product per head, so EVERY layer's entropy, per-key
scores and row normalisers are compared with it.  Phase B is checked in full where the oracle can
afford it: the selection of every KV head of four layers (largest, smallest and two middle budgets),
and, for one head of the layer with the largest budget and of a layer on the small-budget arg-max
kernel, every arg-max target (the oracle's similarity evaluated block by block) and every merged
slot.  Properties that hold at any size (every token accounted for, ascending indices, the recent
window kept, bit-identical reruns) are checked for all layers and heads."""
from concurrent.futures import ThreadPoolExecutor

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


def _oracle_phase_a(q, k, mod):
    """(entropy, scores, row_stats) of one layer from the oracle, on the bits the device saw."""
    qh, kh = P.np64(q), P.np64(k)
    return O.cross_modal_entropy(qh, kh, mod), O.window_scores(qh, kh), O.row_stats(qh, kh, mod)


def _detail_layers(budgets, n, small_max):
    """Layers whose phase B is compared in detail: the largest budget that still merges something, the
    smallest, two in between, and (when there is one) the largest budget that the small-budget arg-max
    kernel serves."""
    S = budgets[:, 0]
    merging = [int(l) for l in np.argsort(-S, kind="stable") if S[l] < n]
    picks = [merging[0], merging[-1], merging[len(merging) // 3], merging[(2 * len(merging)) // 3]]
    small = [l for l in merging if S[l] <= small_max]
    large = [l for l in merging if S[l] > small_max]
    full = [merging[0]]
    if small:
        picks.append(small[0])
        full.append(small[0])
    if large and large[-1] not in full:
        full.append(large[-1])                     # the smallest budget on the row-gathering kernel
        picks.append(large[-1])
    return sorted(set(picks)), full


@pytest.mark.parametrize("name", ["multi_image_8k", "long_video_19k", "multimodal_32k", "long_video_128k"])
def test_full_size_pass_against_the_oracle(name, parity_report):
    from paper_2502_17599_b200.binding import NEAREST_SMALL_MAX_S
    from paper_2502_17599_b200.pipeline import CompressionPass
    wl = W.WORKLOADS[name]
    n, L, hkv, d = wl.n_tokens, wl.n_layers, wl.n_kv_heads, wl.head_dim
    mod = wl.modality().numpy()
    qs, ks, vs = [], [], []
    for l in range(L):
        q, k, v = W.make_layer(wl, l, "cuda")
        qs.append(q); ks.append(k); vs.append(v)
    cp = CompressionPass(wl)
    cp.run(qs, ks, vs)
    cp.check()

    # ---- a second run of the same pass gives the same bits everywhere (no float atomics, no races)
    first = [t.clone() for t in (cp.entropy, cp.budgets, cp.scores)]
    live = lambda: [torch.cat([x[l, :, : int(cp.budgets[l, 0])].reshape(-1).view(torch.uint8) for l in range(L)])
                    for x in (cp.k_out, cp.v_out, cp.counts, cp.idx_c)]
    first_live = live()
    cp.run(qs, ks, vs)
    cp.check()
    for a, b_ in zip(first, (cp.entropy, cp.budgets, cp.scores)):
        assert torch.equal(a, b_)
    for a, b_ in zip(first_live, live()):
        assert torch.equal(a, b_)
    del first, first_live

    # ---- phase A of EVERY layer against the oracle: entropy, per-key scores, row normalisers
    ent = P.np64(cp.entropy)
    buf = P.GpuBuffers(wl)
    a_or = {}
    with ThreadPoolExecutor(max_workers=4) as pool:
        jobs = [pool.submit(_oracle_phase_a, qs[l], ks[l], mod) for l in range(L)]
        for l in range(L):
            # the same call outside the pass, to see the layer's normalisers: same kernels, same bits
            cp.ctx.window_scores(l, qs[l], ks[l], buf.row_stats, buf.scores, buf.entropy)
            cp.ctx.check()
            assert torch.equal(buf.scores, cp.scores[l]) and float(buf.entropy[l]) == float(cp.entropy[l])
            want_e, want_a, want_rs = jobs[l].result()
            jobs[l] = None
            P.assert_entropy_close(ent[l], want_e)
            P.assert_scores_close(P.np64(cp.scores[l]), want_a)
            P.assert_row_stats_close(P.np64(buf.row_stats), want_rs)
            a_or[l] = want_a

    # ---- budgets: bit-exact from the entropies the device produced; they sum to the global budget
    budgets = cp.budgets.cpu().numpy()
    np.testing.assert_array_equal(budgets, O.allocate_budgets(ent, wl.global_budget, n, wl.min_budget))
    assert int(budgets[:, 0].sum()) == wl.global_budget
    assert (ent >= 0).all() and (ent <= np.log((mod == 1).sum()) + 1e-4).all()

    # ---- properties of every layer and head
    for l in range(L):
        S, M, N = (int(x) for x in budgets[l])
        idx = cp.idx_c[l, :, :S].cpu().numpy()
        cnt = cp.counts[l, :, :S].cpu().numpy()
        assert (np.diff(idx, axis=1) > 0).all() and idx.min() >= 0 and idx.max() == n - 1
        assert (idx[:, S - M:] == np.arange(n - M, n)[None, :]).all()          # the recent window is kept
        assert (cnt >= 1).all() and (cnt.sum(axis=1) == n).all()               # every token is kept or merged
        sc = cp.scores[l].sum(dim=1).cpu().numpy()
        np.testing.assert_allclose(sc, (wl.n_q_heads // hkv) * wl.window, rtol=2e-4)

    # ---- phase B in detail
    detail, full = _detail_layers(budgets, n, NEAREST_SMALL_MAX_S if (wl.dtype == "bf16" and d == 128) else 0)
    swaps = ties = ulp_used = 0
    checked_rows = checked_slots = 0
    for layer in detail:
        S, M, N = (int(x) for x in budgets[layer])
        # the layer through the separate entry points, to see the less-important list and the targets
        cp.ctx.select_topk(layer, cp.scores[layer], cp.budgets, buf.idx_c, buf.idx_less, buf.cap)
        cp.ctx.merge_kv(layer, ks[layer], vs[layer], cp.budgets, buf.idx_c, buf.idx_less, buf.k_out, buf.v_out,
                        buf.counts, buf.target, buf.cap)
        cp.ctx.check()
        assert torch.equal(buf.idx_c[:, :S], cp.idx_c[layer, :, :S])
        assert torch.equal(buf.k_out[:, :S], cp.k_out[layer, :, :S]) and torch.equal(buf.v_out[:, :S], cp.v_out[layer, :, :S])
        assert torch.equal(buf.counts[:, :S], cp.counts[layer, :, :S])
        for g in range(hkv):                       # selection of every KV head against the oracle's scores
            cons = buf.idx_c[g, :S].cpu().numpy().astype(np.int64)
            less = buf.idx_less[g, : n - S].cpu().numpy().astype(np.int64)
            swaps += P.compare_selection(cons, a_or[layer][g], mod, M, N)
            np.testing.assert_array_equal(less, np.setdiff1d(np.arange(n), cons))
        if layer not in full or S >= n:
            continue
        g = (layer * 7 + 1) % hkv                  # one head per layer, not always the first
        kh, vh = P.np64(ks[layer][g]), P.np64(vs[layer][g])
        cons = buf.idx_c[g, :S].cpu().numpy().astype(np.int64)
        less = buf.idx_less[g, : n - S].cpu().numpy().astype(np.int64)
        tgt = buf.target[g, : n - S].cpu().numpy().astype(np.int64)
        ties += P.compare_targets_blockwise(tgt, kh, cons, less)                # every less-important row
        st = P.compare_merged(P.np64(buf.k_out[g, :S]), P.np64(buf.v_out[g, :S]), buf.counts[g, :S].cpu().numpy(),
                              kh, vh, cons, less, tgt, wl.dtype)                # every merged slot
        ulp_used += st["ulp_allowance_used"]
        checked_rows += less.size
        checked_slots += S
    parity_report(f"{name}: phase A of all {L} layers in tolerance; selection of all {hkv} heads of layers {detail}: "
                  f"{swaps} tolerated swaps; layers {full} (one head each): {checked_rows} arg-max rows with {ties} "
                  f"tolerated near-ties, {checked_slots} merged slots with {ulp_used} elements on the one-ulp allowance")
    cp.close()


def test_full_size_variants_ablation_modes_vision_to_text_term_and_decoding_step():
    """The long-video 18.9K configuration at full size: the ablation modes of Table 5 (uniform budgets,
    eviction instead of merging, mean of per-head entropies), the E_VT term with a window of visual query
    rows, and one decoding step over the compressed cache of a layer, each against the oracle."""
    from paper_2502_17599_b200.pipeline import CompressionPass
    wl = W.WORKLOADS["long_video_19k"]
    n, L, hkv = wl.n_tokens, wl.n_layers, wl.n_kv_heads
    mod = wl.modality().numpy()
    qs, ks, vs = [], [], []
    for l in range(L):
        q, k, v = W.make_layer(wl, l, "cuda")
        qs.append(q); ks.append(k); vs.append(v)

    # ---- Table 5's ablation rows: no dynamic allocation, no merging; and per-head entropies
    cp = CompressionPass(wl, entropy_mode=1, alloc_mode=1, merge_mode=1)
    cp.run(qs, ks, vs)
    cp.check()
    budgets = cp.budgets.cpu().numpy()
    ent = P.np64(cp.entropy)
    np.testing.assert_array_equal(budgets, O.allocate_budgets(ent, wl.global_budget, n, wl.min_budget, alloc_mode=1))
    assert budgets[:, 0].max() - budgets[:, 0].min() <= 1 and int(budgets[:, 0].sum()) == wl.global_budget
    layer = L // 2
    qh = P.np64(qs[layer])
    kh = np.stack([P.np64(ks[layer][g]) for g in range(hkv)])
    P.assert_entropy_close(ent[layer], O.cross_modal_entropy(qh, kh, mod, entropy_mode=1))
    S = int(budgets[layer, 0])
    idx = cp.idx_c[layer, :, :S].long()
    assert (cp.counts[layer, :, :S] == 1).all()
    for g in range(hkv):
        assert torch.equal(cp.k_out[layer, g, :S], ks[layer][g][idx[g]]) and torch.equal(cp.v_out[layer, g, :S], vs[layer][g][idx[g]])
    cp.close()

    # ---- the paper's modes: E_CM with the vision-to-text term, then one decoding step over the result
    cp = CompressionPass(wl)
    cp.run(qs, ks, vs)
    cp.check()
    n_rows = 32
    qv, pos = W.make_visual_queries(wl, layer, n_rows, "cuda")
    ent_full = cp.entropy.clone()
    cp.ctx.layer_entropy(layer, None, ks[layer], None, ent_full, q_vis=qv, q_vis_pos=pos, n_vis_rows=n_rows)
    cp.check()
    want = O.cross_modal_entropy(qh, kh, mod, q_vis=P.np64(qv), q_vis_pos=pos.cpu().numpy().astype(np.int64))
    P.assert_entropy_close(float(ent_full[layer]), want)
    assert float(ent_full[layer]) > float(cp.entropy[layer])          # -E_VT is a positive addition

    S = int(cp.budgets[layer, 0])
    q_new = qs[layer][:, -1, :].contiguous()
    out = torch.zeros((wl.n_q_heads, wl.head_dim), dtype=torch.float32, device="cuda")
    cp.ctx.decode_attention(layer, q_new, cp.k_out[layer], cp.v_out[layer], out, budgets=cp.budgets)
    cp.check()
    want_out = O.decode_attention(P.np64(q_new), P.np64(cp.k_out[layer, :, :S]), P.np64(cp.v_out[layer, :, :S]))
    np.testing.assert_allclose(P.np64(out), want_out, rtol=1e-4, atol=1e-4)
    cp.close()


def test_one_prompt_sharded_by_layer_gives_the_unsharded_results():
    """The layer-sharded pass (one prompt, layers dealt round-robin to ranks, entropies exchanged between the
    phases) emulated on one GPU: two shards run one after the other, each receiving the other's entropies through
    the exchange hook.  Budgets and every owned layer's outputs equal the unsharded pass bit for bit."""
    from paper_2502_17599_b200.pipeline import CompressionPass, owned_layers
    wl = W.WORKLOADS["long_video_19k"].with_(name="long_video_19k_6l", n_layers=6)
    L = wl.n_layers
    qs, ks, vs = [], [], []
    for l in range(L):
        q, k, v = W.make_layer(wl, l, "cuda")
        qs.append(q); ks.append(k); vs.append(v)
    whole = CompressionPass(wl, n_streams=2)
    whole.run(qs, ks, vs)
    whole.check()
    for rank in range(2):
        mine = owned_layers(L, rank, 2)
        others = torch.zeros_like(whole.entropy)
        for l in range(L):
            if l not in mine:
                others[l] = whole.entropy[l]
        part = CompressionPass(wl, n_streams=2)
        part.run([q if l in mine else None for l, q in enumerate(qs)], ks, vs, layer_shard=(rank, 2),
                 exchange=lambda e: e.add_(others))
        part.check()
        assert torch.equal(part.entropy, whole.entropy) and torch.equal(part.budgets, whole.budgets)
        for l in mine:
            S = int(whole.budgets[l, 0])
            assert torch.equal(part.scores[l], whole.scores[l])
            assert torch.equal(part.idx_c[l, :, :S], whole.idx_c[l, :, :S])
            assert torch.equal(part.counts[l, :, :S], whole.counts[l, :, :S])
            assert torch.equal(part.k_out[l, :, :S], whole.k_out[l, :, :S])
            assert torch.equal(part.v_out[l, :, :S], whole.v_out[l, :, :S])
        part.close()
    whole.close()
