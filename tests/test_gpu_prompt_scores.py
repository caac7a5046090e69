"""GPU parity of Eq. 8 taken over every prompt row (meda_prompt_scores: the column sums of the whole causal
attention matrix) against the oracle's window_scores with the window equal to the prompt."""
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


def make_ctx(wl, **kw):
    from paper_2502_17599_b200 import binding
    return binding.Context.for_workload(wl, **kw)


def prompt_cases():
    long_spans = W._spans((37, 0), (45 * 61, 1), (75, 0))                    # 2,857 tokens: 12 row blocks, ragged tail
    return [
        W.WORKLOADS["tiny"],                                                 # fp32, d = 64: CUDA-core blocks of 64 rows
        W.small_variant("small_mha_d64", n_q_heads=4, n_kv_heads=4, head_dim=64, window=17, seed=2),
        W.small_variant("small_f32_gqa", dtype="f32", n_q_heads=4, n_kv_heads=2, head_dim=128, seed=3),
        W.small_variant(),                                                   # bf16, d = 128, GQA 3:1, n = 661: tensor cores
        W.small_variant("prompt_2857", spans=long_spans, seed=6),
        W.small_variant("prompt_512", spans=((0, 40, 0), (40, 480, 1), (480, 512, 0)), frame_tokens=0, seed=7),
        W.small_variant("prompt_97", spans=((0, 11, 0), (11, 70, 1), (70, 97, 0)), frame_tokens=0, rho=0.4, seed=8),
        W.small_variant("prompt_129_mha", spans=((0, 100, 1), (100, 129, 0)), n_q_heads=2, n_kv_heads=2,
                        frame_tokens=0, rho=0.4, seed=9),
    ]


def scratch_for(ctx):
    nbytes = ctx.prompt_scores_scratch_bytes()
    return torch.empty(nbytes, dtype=torch.uint8, device="cuda") if nbytes else None


@pytest.mark.parametrize("wl", prompt_cases(), ids=lambda w: w.name)
def test_prompt_scores_match_the_oracle_with_the_window_equal_to_the_prompt(wl):
    n, group = wl.n_tokens, wl.n_q_heads // wl.n_kv_heads
    ctx = make_ctx(wl)
    scratch = scratch_for(ctx)
    for layer in range(min(2, wl.n_layers)):
        _, k, _ = W.make_layer(wl, layer, "cuda")
        q_all = W.make_prompt_queries(wl, layer, "cuda")
        scores = torch.full((wl.n_kv_heads, n), -7.0, dtype=torch.float32, device="cuda")
        ctx.prompt_scores(q_all, k, scores, scratch)
        ctx.check()
        qh, kh = P.np64(q_all), P.np64(k)
        want = O.window_scores(qh, kh)                       # the window is the whole prompt: Eq. 8 as printed
        got = P.np64(scores)
        P.assert_scores_close(got, want)
        np.testing.assert_allclose(got.sum(axis=1), group * n, rtol=1e-5)    # every row is a distribution
        # a second call gives the same bits
        again = torch.zeros_like(scores)
        ctx.prompt_scores(q_all, k, again, scratch)
        ctx.check()
        assert torch.equal(again, scores)
    ctx.close()


def test_prompt_scores_feed_the_selection_and_reject_a_small_scratch():
    from paper_2502_17599_b200 import binding
    wl = W.small_variant("prompt_select", window=32, seed=11)
    n = wl.n_tokens
    ctx = make_ctx(wl)
    buf = P.GpuBuffers(wl)
    mod = wl.modality().numpy()
    _, k, _ = W.make_layer(wl, 0, "cuda")
    q_all = W.make_prompt_queries(wl, 0, "cuda")
    need = ctx.prompt_scores_scratch_bytes()
    assert need >= wl.n_q_heads * n * 20
    with pytest.raises(binding.MedaError) as err:
        ctx.prompt_scores(q_all, k, buf.scores, torch.empty(need - 16, dtype=torch.uint8, device="cuda"))
    assert err.value.status == binding.MEDA_ERR_WORKSPACE
    with pytest.raises(binding.MedaError):
        ctx.prompt_scores(q_all, k, buf.scores, None)
    ctx.prompt_scores(q_all, k, buf.scores, scratch_for(ctx))
    S = n // 4
    M = (3 * S) // 4
    budgets = torch.tensor([[S, M, S - M]] * wl.n_layers, dtype=torch.int32, device="cuda")
    ctx.select_topk(0, buf.scores, budgets, buf.idx_c, buf.idx_less, buf.cap)
    ctx.check()
    a_s = O.window_scores(P.np64(q_all), P.np64(k))
    for g in range(wl.n_kv_heads):
        P.compare_selection(buf.idx_c[g, :S].cpu().numpy(), a_s[g], mod, M, S - M)
    ctx.close()


@pytest.mark.parametrize("name,kv_heads", [("multi_image_8k", (0, 31)), ("long_video_19k", (2,))])
def test_prompt_scores_at_full_size_on_sampled_heads(name, kv_heads):
    """One layer of a benchmark configuration: every KV head is checked for what holds at any size (the scores
    of a head sum to group * n); the KV heads named are compared with the oracle key by key."""
    wl = W.WORKLOADS[name]
    n, group = wl.n_tokens, wl.n_q_heads // wl.n_kv_heads
    ctx = make_ctx(wl)
    scratch = scratch_for(ctx)
    layer = 1
    _, k, _ = W.make_layer(wl, layer, "cuda")
    q_all = W.make_prompt_queries(wl, layer, "cuda")
    scores = torch.zeros((wl.n_kv_heads, n), dtype=torch.float32, device="cuda")
    ctx.prompt_scores(q_all, k, scores, scratch)
    ctx.check()
    got = P.np64(scores)
    assert (got > 0).all()
    np.testing.assert_allclose(got.sum(axis=1), group * n, rtol=1e-5)
    for g in kv_heads:
        qh = P.np64(q_all[g * group:(g + 1) * group])
        kh = P.np64(k[g:g + 1])
        want = P.oracle_prompt_scores(qh, kh)
        P.assert_scores_close(got[g:g + 1], want)
    again = torch.zeros_like(scores)
    ctx.prompt_scores(q_all, k, again, scratch)
    ctx.check()
    assert torch.equal(again, scores)
    ctx.close()
