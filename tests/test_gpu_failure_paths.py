"""Device-side failure reporting, exercised without faulting or hanging anything: the bounded wait
that every tensor-core pipeline of the library uses is made to run out by a self-test kernel that
waits on a barrier nothing arrives on, with a limit of a few thousand cycles."""
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


def test_a_wait_that_runs_out_is_reported_once_and_the_context_keeps_working():
    from paper_2502_17599_b200 import binding as B
    wl = W.small_variant("tc_w32_timeout", window=32, seed=4)       # takes the tensor-core phase-A kernels
    ctx = B.Context.for_workload(wl)
    buf = P.GpuBuffers(wl)
    mod = wl.modality().numpy()
    (q, k, v), (qh, kh, vh) = P.layer_inputs(wl, 0, "cuda")

    assert ctx.poll_status() == B.MEDA_OK
    ctx.selftest_wait_timeout(5000)
    assert ctx.poll_status() == B.MEDA_ERR_TIMEOUT                   # recorded in the status word ...
    assert ctx.poll_status() == B.MEDA_OK                            # ... and cleared by the poll
    # the first error wins: a second timeout before the poll still reads as one
    ctx.selftest_wait_timeout(2000)
    ctx.selftest_wait_timeout(2000)
    with pytest.raises(B.MedaError) as err:
        ctx.check()
    assert err.value.status == B.MEDA_ERR_TIMEOUT
    # the context is as usable as before: an ordinary call on it still matches the oracle
    ctx.window_scores(0, q, k, buf.row_stats, buf.scores, buf.entropy)
    ctx.check()
    P.assert_entropy_close(float(buf.entropy[0]), O.cross_modal_entropy(qh, kh, mod))
    P.assert_scores_close(P.np64(buf.scores), O.window_scores(qh, kh))
    # bad limits are refused on the host
    for cycles in (0, -5, 3_000_000_000):
        with pytest.raises(B.MedaError) as err:
            ctx.selftest_wait_timeout(cycles)
        assert err.value.status == B.MEDA_ERR_INVALID_ARG
    ctx.close()
