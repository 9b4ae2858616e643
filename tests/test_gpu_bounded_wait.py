"""The waits of the staged kernels are bounded: a wait that can never succeed ends by its poll limit,
the kernel says so and returns, and the context keeps working.  The library's self-test runs the
very wait routine on a barrier that nothing completes (limit 1024 polls)."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import codes_np, drifting_grads, make_ctx, same_values, to_np
from paper_1901_08227_b200 import tng

pytestmark = pytest.mark.gpu


def test_a_wait_that_cannot_succeed_gives_up_and_the_context_stays_usable():
    d, M, K = 2048 * 9 + 100, 3, 2
    ctx = make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_DIFF, seed_lo=2)
    orc = oracle.State(d, M, K, tng.CODEC_TERN2, tng.NORM_DIFF, seed_lo=2)
    out = torch.empty(d, device="cuda")
    grads = list(drifting_grads(1, 4, M, d, "cuda"))
    for g in grads[:2]:
        ctx.step(g, out)
        orc.step(to_np(g))
    assert ctx.selftest_bounded_wait() is True
    st = ctx.stats()
    assert st.pipeline_error == 0                       # the self-test does not touch the context's error word
    for g in grads[2:]:                                 # ... and the rounds go on, bit for bit
        ctx.step(g, out)
        want = orc.step(to_np(g))
        assert np.array_equal(codes_np(ctx.wire()[0]), orc.codes())
        assert same_values(to_np(out), want)
    assert ctx.stats().rounds == 4
