"""Helpers shared by the GPU parity tests: running the CUDA path through the C-ABI binding,
running the oracle on the same bits, and the comparison rules.

Comparison rules and tolerances:
  budgets          bit-exact
  selected sets    bit-exact except swaps between candidates whose ORACLE scores differ by less
                   than 1e-5 relative; swaps are counted and returned
  entropies        1e-4 relative
  arg-max targets  exact except where the oracle's similarity of the GPU's choice is within 1e-5
                   of the oracle's maximum; counted and returned
  merged K/V       against the oracle re-run with the GPU's (validated) index sets and targets:
                   bf16: 2e-2 max-abs after rounding the oracle to bf16, one bf16 ulp where |x| >= 8;
                   fp32: 1e-5 relative (+1e-6 absolute)
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import meda_oracle as O

SWAP_RTOL = 1e-5
ENTROPY_RTOL = 1e-4
TARGET_ATOL = 1e-5
MERGE_BF16_ATOL = 2e-2
MERGE_F32_RTOL = 1e-5


def np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def layer_inputs(wl, layer, device):
    """Generates one layer once on `device` and returns (device tensors, the same bits as fp64 numpy)."""
    from paper_2502_17599_b200 import workloads as W
    q, k, v = W.make_layer(wl, layer, device)
    return (q, k, v), (np64(q), np64(k), np64(v))


class GpuBuffers:
    """Device buffers of one context's phase A / phase B calls."""

    def __init__(self, wl, cap=None, device="cuda"):
        n, hkv, hq, w, d = wl.n_tokens, wl.n_kv_heads, wl.n_q_heads, wl.window, wl.head_dim
        self.cap = n if cap is None else cap
        self.row_stats = torch.zeros((hq, w, 4), dtype=torch.float32, device=device)
        self.scores = torch.zeros((hkv, n), dtype=torch.float32, device=device)
        self.entropy = torch.zeros(wl.n_layers, dtype=torch.float32, device=device)
        self.budgets = torch.zeros((wl.n_layers, 3), dtype=torch.int32, device=device)
        self.idx_c = torch.full((hkv, self.cap), -1, dtype=torch.int32, device=device)
        self.idx_less = torch.full((hkv, n), -1, dtype=torch.int32, device=device)
        self.k_out = torch.zeros((hkv, self.cap, d), dtype=wl.torch_dtype, device=device)
        self.v_out = torch.zeros((hkv, self.cap, d), dtype=wl.torch_dtype, device=device)
        self.counts = torch.zeros((hkv, self.cap), dtype=torch.int32, device=device)
        self.target = torch.full((hkv, n), -1, dtype=torch.int32, device=device)


# ----------------------------------------------------------------------------- comparisons

def assert_entropy_close(got: float, want: float):
    assert abs(got - want) <= ENTROPY_RTOL * max(abs(want), 1e-12), (got, want)


def assert_row_stats_close(got: np.ndarray, want: np.ndarray):
    """Compares the log-normalisers m + ln z (the quantity the softmax depends on) and the maxima."""
    for a, b in ((0, 1), (2, 3)):
        live = want[..., b] > 0
        assert ((got[..., b] > 0) == live).all()
        if not live.any():
            continue
        lse_g = got[..., a][live] + np.log(got[..., b][live])
        lse_w = want[..., a][live] + np.log(want[..., b][live])
        np.testing.assert_allclose(lse_g, lse_w, rtol=0, atol=2e-5 * np.maximum(1.0, np.abs(lse_w)).max())
        np.testing.assert_allclose(got[..., a][live], want[..., a][live], rtol=2e-5, atol=2e-5)


def assert_scores_close(got: np.ndarray, want: np.ndarray, rtol=1e-4):
    np.testing.assert_allclose(got, want, rtol=rtol, atol=1e-9)


def compare_selection(gpu_conserved: np.ndarray, a_s: np.ndarray, modality: np.ndarray, n_recent: int, n_important: int) -> int:
    """Checks the GPU's conserved list for one head against the oracle run on the same scores.
    Returns the number of tolerated swaps."""
    want_c, _ = O.select_topk(a_s, modality, n_recent, n_important)
    got = np.asarray(gpu_conserved, dtype=np.int64)
    assert got.size == want_c.size
    assert (np.diff(got) > 0).all(), "conserved indices must be strictly ascending"
    only_or = np.setdiff1d(want_c, got)
    only_gpu = np.setdiff1d(got, want_c)
    assert only_or.size == only_gpu.size
    if only_or.size == 0:
        return 0
    n = a_s.size
    n_cand = n - n_recent
    assert (only_gpu < n_cand).all() and (only_or < n_cand).all()
    # a swap is allowed only inside one modality class and only between scores within 1e-5 relative
    for cls in (O.TEXT, O.VISUAL):
        a = only_or[modality[only_or] == cls]
        b = only_gpu[modality[only_gpu] == cls]
        assert a.size == b.size, "swap across the text/visual boundary"
        if a.size == 0:
            continue
        lo = min(a_s[a].min(), a_s[b].min())
        hi = max(a_s[a].max(), a_s[b].max())
        assert hi - lo <= SWAP_RTOL * max(hi, 1e-300), (lo, hi)
    return int(only_or.size)


def compare_targets(gpu_target: np.ndarray, k_g: np.ndarray, conserved: np.ndarray, less: np.ndarray) -> int:
    """Checks the GPU's nearest-slot choice for one head.  Returns the number of tolerated near-ties."""
    want, u = O.nearest_conserved(k_g, conserved, less)
    got = np.asarray(gpu_target, dtype=np.int64)
    assert got.shape == want.shape
    if got.size == 0:
        return 0
    assert got.min() >= 0 and got.max() < conserved.size
    diff = np.nonzero(got != want)[0]
    if diff.size:
        chosen = u[diff, got[diff]]
        best = u[diff, want[diff]]
        assert (best - chosen <= TARGET_ATOL).all(), float((best - chosen).max())
    return int(diff.size)


def compare_targets_blockwise(gpu_target: np.ndarray, k_g: np.ndarray, conserved: np.ndarray, less: np.ndarray,
                              block: int = 1024, threads: int = 4) -> int:
    """compare_targets for a head whose similarity matrix does not fit memory at once: the oracle's
    cosine_similarity is evaluated on consecutive blocks of `block` less-important rows against ALL
    conserved keys (the arg-max of a row needs nothing from other rows), so every row is still checked
    against the oracle's own arithmetic.  Blocks are independent; a few run at a time on host threads.
    Returns the number of tolerated near-ties."""
    from concurrent.futures import ThreadPoolExecutor
    got = np.asarray(gpu_target, dtype=np.int64)
    assert got.shape == (less.size,)
    if got.size == 0:
        return 0
    assert got.min() >= 0 and got.max() < conserved.size
    k_c = k_g[conserved]

    def one(p0: int) -> int:
        rows = slice(p0, min(p0 + block, less.size))
        u = O.cosine_similarity(k_g[less[rows]], k_c)
        want = np.argmax(u, axis=1)
        diff = np.nonzero(got[rows] != want)[0]
        if diff.size:
            gap = u[diff, want[diff]] - u[diff, got[rows][diff]]
            assert (gap <= TARGET_ATOL).all(), (p0, float(gap.max()))
        return int(diff.size)

    with ThreadPoolExecutor(max_workers=threads) as pool:
        return int(sum(pool.map(one, range(0, less.size, block))))


def compare_merged(got_k, got_v, got_counts, k_g, v_g, conserved, less, target, dtype: str, merge_mode=0) -> dict:
    """Merged rows of one head against the oracle re-run with the GPU's sets and targets."""
    km, vm, counts, _ = O.merge_kv(k_g, v_g, conserved, less, target=np.asarray(target, dtype=np.int64), merge_mode=merge_mode)
    np.testing.assert_array_equal(np.asarray(got_counts, dtype=np.int64), counts)
    stats = dict(max_abs=0.0, ulp_allowance_used=0)
    for got, want in ((got_k, km), (got_v, vm)):
        if dtype == "bf16":
            want_r = O.round_to_bf16(want)
            err = np.abs(got - want_r)
            big = np.abs(want_r) >= 8.0
            ulp = np.where(big, 2.0 ** (np.floor(np.log2(np.maximum(np.abs(want_r), 1e-30))) - 7), 0.0)
            ok = (err <= MERGE_BF16_ATOL) | (big & (err <= ulp))
            assert ok.all(), float(err.max())
            stats["ulp_allowance_used"] += int((big & (err > MERGE_BF16_ATOL)).sum())
            stats["max_abs"] = max(stats["max_abs"], float(err.max()) if err.size else 0.0)
            # unmerged slots are copies of the input rows
            single = counts == 1
            np.testing.assert_array_equal(got[single], want[single])
        else:
            err = np.abs(got - want)
            assert (err <= MERGE_F32_RTOL * np.abs(want) + 1e-6).all(), float(err.max())
            stats["max_abs"] = max(stats["max_abs"], float(err.max()) if err.size else 0.0)
    return stats


def oracle_prompt_scores(q_all: np.ndarray, k: np.ndarray, block: int = 1024) -> np.ndarray:
    """Eq. 8 over every prompt row with the oracle: its window_scores evaluated on consecutive blocks of
    query rows at their own positions and added up (the score is a sum over rows), so that the n x n
    matrix never has to exist at once.  q_all [Hq, n, d], k [Hkv, n, d] -> [Hkv, n]."""
    n = k.shape[1]
    out = np.zeros((k.shape[0], n))
    for p0 in range(0, n, block):
        pos = np.arange(p0, min(p0 + block, n))
        out[:, : pos[-1] + 1] += O.window_scores(q_all[:, pos], k[:, : pos[-1] + 1], q_pos=pos)
    return out
