"""meda_row_stats_static: the entry point for callers that cannot allocate device memory.

Some users of this library run inside a process that gave all of device memory to its own pool at
start-up, or call from a section that must not stall on the device-wide synchronisation of
cudaMalloc / cudaFree; they cannot create a context.  The static entry point serves them from a
fixed scratch array in the library's device image.  The GPU test calls it through the C ABI twice in
a row, on different inputs, and compares each result with what the ordinary, context-based entry
point (meda_window_scores) writes for the same inputs; the second call also shows that what the first
one left in the shared scratch array does no harm.  This file sorts after the other test files on
purpose, so a run that stops at the first failure has already been through all of them.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2502_17599_b200 import workloads as W


@pytest.fixture(scope="module")
def B():
    from paper_2502_17599_b200 import build, binding
    build.build()
    binding.load_library()
    return binding


def test_static_entry_point_rejects_bad_sizes_without_a_device(B):
    lib = B.load_library()
    one = ctypes.c_void_p(256)        # never dereferenced: every call below fails its argument checks first
    call = lambda hq, hkv, d, n, w, dt: lib.meda_row_stats_static(one, one, one, hq, hkv, d, n, w, dt, one, None)
    assert call(64, 8, 128, 10000, 128, B.MEDA_BF16) == B.MEDA_ERR_SHAPE      # 8192 rows > the fixed scratch
    assert call(33, 1, 128, 10000, 128, B.MEDA_BF16) == B.MEDA_ERR_SHAPE      # 4224 rows
    assert call(4, 3, 128, 1000, 32, B.MEDA_BF16) == B.MEDA_ERR_SHAPE
    assert call(4, 2, 96, 1000, 32, B.MEDA_BF16) == B.MEDA_ERR_SHAPE
    assert call(4, 2, 128, 16, 32, B.MEDA_BF16) == B.MEDA_ERR_SHAPE           # window > n_tokens
    assert call(4, 2, 128, 1000, 32, 7) == B.MEDA_ERR_INVALID_ARG
    assert lib.meda_row_stats_static(None, one, one, 4, 2, 128, 1000, 32, 0, one, None) == B.MEDA_ERR_INVALID_ARG


@pytest.mark.gpu
@pytest.mark.parametrize("wl", [
    W.small_variant(),                                                 # bf16, window 24: both entry points run the same kernels
    W.small_variant("static_tc_w32", window=32, seed=4),               # bf16, window 32: the context takes the tensor-core kernels
    W.small_variant("static_f32", dtype="f32", n_q_heads=4, n_kv_heads=2, head_dim=64, seed=3),
], ids=lambda w: w.name)
def test_static_entry_point_matches_the_context_path_twice_in_a_row(B, wl):
    import parity as P
    ctx = B.Context.for_workload(wl)
    buf = P.GpuBuffers(wl)
    modality = wl.modality("cuda")
    got = torch.full_like(buf.row_stats, float("nan"))
    for call, layer in enumerate((0, 1)):
        (q, k, v), _ = P.layer_inputs(wl, layer, "cuda")
        ctx.window_scores(layer, q, k, buf.row_stats, buf.scores, None)
        ctx.check()
        got.fill_(float("nan"))
        B.row_stats_static(q, k, modality, got)
        torch.cuda.synchronize()
        want = P.np64(buf.row_stats)
        have = P.np64(got)
        assert np.isfinite(have[..., 1]).all(), f"call {call}: output not fully written"
        # the tolerance the parity tests use for row normalisers (log-sum-exp within 2e-5)
        P.assert_row_stats_close(have, want)
        if not (wl.dtype == "bf16" and wl.head_dim == 128 and wl.window in (32, 64)):
            np.testing.assert_array_equal(have, want)      # same kernels on both sides: same bits
    ctx.close()
