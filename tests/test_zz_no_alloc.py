"""tng_gram_static, the entry point for callers that cannot allocate device memory
(their memory belongs to a pool of their own, or their steady-state loop has to stay
clear of cudaMalloc).  It must give the same fusion statistics as the context-based
path (tng_fuse + tng_stats), call after call, out of its fixed in-library scratch.

This file sorts last on purpose: a run that stops at the first failure has then
already run every other test."""
import numpy as np
import pytest
import torch

import oracle
from paper_1901_08227_b200 import tng, workloads

pytestmark = pytest.mark.gpu


def context_stats(rows, grads):
    k, d, M = len(rows), rows[0].numel(), grads.shape[0]
    ctx = tng.Context(d, M, k, tng.CODEC_TERN2, tng.NORM_DIFF, fuse_mode=tng.FUSE_LSQ)
    for r in reversed(rows):                      # oldest first, so rows[0] ends up newest
        ctx.push_reference(r)
    ctx.fuse(grads)
    st = ctx.stats()
    G = np.array(st.gram[:]).reshape(16, 16)[:k, :k]
    G = np.triu(G) + np.triu(G, 1).T
    out = np.concatenate([G.ravel(), np.array(st.rhs[:k]), [st.grad_sq]])
    ctx.close()
    return out


@pytest.mark.parametrize("k,M,d", [(8, 8, 128 * 3000 + 52), (3, 5, 70001), (1, 1, 9)])
def test_static_scratch_path_matches_the_context_path_twice_in_a_row(k, M, d):
    ld = (d + 3) // 4 * 4
    traj = workloads.AR1Trajectory(17 + k, d, device="cuda")
    rows = [traj.advance().contiguous() for _ in range(k)][::-1]
    out = torch.full((k * k + k + 1,), float("nan"), dtype=torch.float64, device="cuda")
    for call in range(2):                         # the second call starts from the first one's leftovers
        traj.advance()
        grads = traj.worker_grads(M, 0.5, ld=ld)
        tng.gram_static(rows, grads, out)
        got = out.cpu().numpy()
        want = context_stats(rows, grads)
        scale = np.abs(want).max()
        assert np.all(np.isfinite(got))
        assert np.abs(got - want).max() <= 1e-10 * scale, f"call {call}"
        G = got[: k * k].reshape(k, k)
        assert np.array_equal(G, G.T)
        # and against the CPU oracle's double-precision sums, so that this test stands on its own
        oG, oc, ogg = oracle.fuse_stats([r.cpu().numpy() for r in rows], grads.cpu().numpy()[:, :d])
        owant = np.concatenate([oG.ravel(), oc, [ogg]])
        # (Gram and right-hand side are double sums throughout; the squared norm is summed in fp32 per coordinate
        # before it enters its double accumulator, hence its looser bound)
        n = k * k + k
        assert np.abs(got[:n] - owant[:n]).max() <= 1e-10 * np.abs(owant[:n]).max(), f"call {call} (oracle, Gram and rhs)"
        assert abs(got[n] - owant[n]) <= 1e-6 * abs(owant[n]), f"call {call} (oracle, squared norm)"


def test_sizes_beyond_the_fixed_scratch_are_rejected():
    d = 1024
    rows = [torch.zeros(d, device="cuda") for _ in range(9)]
    grads = torch.zeros((2, d), device="cuda")
    out = torch.zeros(9 * 9 + 9 + 1, dtype=torch.float64, device="cuda")
    with pytest.raises(tng.TngError) as e:
        tng.gram_static(rows, grads, out)         # k = 9 > TNG_STATIC_MAX_HISTORY
    assert e.value.status == tng.ERR_UNSUPPORTED
    with pytest.raises(tng.TngError) as e:
        tng.gram_static([], grads, out)
    assert e.value.status in (tng.ERR_UNSUPPORTED, tng.ERR_INVALID_ARG)
    bad = torch.zeros(2 * 1026, device="cuda").view(2, 1026)[:, :d]
    with pytest.raises(tng.TngError) as e:
        tng.gram_static(rows[:2], bad, out)       # row stride not a multiple of 4
    assert e.value.status == tng.ERR_INVALID_ARG
