"""GPU parity at the benchmark's full size and launch configuration: d = 2^27 coordinates,
M = 8 workers, K = 8 ring entries, quotient form, ternary codes, one scale per 128
coordinates, least-squares fusion -- whole rounds through tng_step, as bench.py times them.

The fusion statistics are global sums, so the oracle computes them on the whole vectors; the
reference, the wire and the aggregate are checked bit for bit on sampled windows of
coordinates (first and last chunks, windows that straddle chunk boundaries, random ones),
which the oracle encodes one by one with the window's coordinate offset."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import rel_l2, to_np
from paper_1901_08227_b200 import tng, workloads

pytestmark = pytest.mark.gpu

D, M, K = 1 << 27, 8, 8


def check_round(ctx, hist, g, out, step, rng):
    """One finished round against the oracle: `hist` are host copies of the ring as it stood before the
    round (newest first), `g` the round's gradient rows, `out` its aggregate, `step` its round number."""
    st = ctx.stats()
    assert st.pipeline_error == 0 and st.solver_fallback == 0 and st.nonfinite_scales == 0
    assert st.rounds == step + 1 and st.k == K
    # ---- fusion statistics and coefficients against the oracle on the whole vectors
    gn = to_np(g)
    oG, oc, ogg = oracle.fuse_stats(hist, gn)
    G = np.array(st.gram[:]).reshape(16, 16)[:K, :K]
    assert rel_l2(G, oG) < 1e-10
    assert rel_l2(np.array(st.rhs[:K]), oc) < 1e-6
    assert st.grad_sq == pytest.approx(ogg, rel=1e-6)
    a64, a32, flag = oracle.fuse_solve(oG, oc, 1e-6)
    assert flag == 0
    alpha = np.array(st.alpha[:K])
    assert np.allclose(alpha, a64, rtol=0, atol=1e-5 * max(1.0, np.abs(a64).max()))
    alpha32 = alpha.astype(np.float32)                # what the combine used

    # ---- reference, wire and aggregate on sampled windows, bit for bit
    ref = ctx.reference()
    codes, scales = ctx.wire()
    newest = ctx.history(0)
    windows = [(0, 2048), (D - 2048, 2048), (2048 * 148 - 256, 512), (2048 * 149 * 7 - 128, 256)]
    windows += [(int(t) * 128, 1024) for t in rng.integers(0, D // 128 - 8, size=60)]
    for i0, n in windows:
        sl = slice(i0, i0 + n)
        want_ref = oracle.combine([h[sl] for h in hist], alpha32)
        got_ref = to_np(ref[sl])
        assert np.array_equal(got_ref.view(np.uint32), want_ref.view(np.uint32)), f"reference differs in window {i0}"
        wc, ws = oracle.encode(np.ascontiguousarray(gn[:, sl]), want_ref, tng.NORM_QUOT, tng.CODEC_TERN2, B=128, seed=(0, 0),
                               t=step, coord_offset=i0)
        t0, t1 = i0 // 128, (i0 + n) // 128
        assert np.array_equal(to_np(codes[:, t0 * 8:t1 * 8]).view(np.uint32), wc), f"codes differ in window {i0}"
        assert np.array_equal(to_np(scales[:, t0:t1]).view(np.uint32), ws.view(np.uint32)), f"scales differ in window {i0}"
        want_out = oracle.decode_aggregate(wc, ws, n, want_ref, tng.NORM_QUOT, tng.CODEC_TERN2, B=128)
        assert np.array_equal(to_np(out[sl]).view(np.uint32), want_out.view(np.uint32)), f"aggregate differs in window {i0}"
        assert np.array_equal(to_np(newest[sl]).view(np.uint32), want_out.view(np.uint32))
    # ---- properties that hold at any size
    assert bool(torch.isfinite(out).all())
    assert bool((scales >= 0).all())


def test_full_size_rounds_in_the_benchmark_configuration():
    """K + 2 rounds.  The first one works on a ring seeded with the stream's means; by the last one every
    ring entry is an aggregate the library decoded itself.  Both are checked against the oracle."""
    free, _ = torch.cuda.mem_get_info()
    if free < 28 * (1 << 30):
        pytest.skip("needs about 28 GiB of free device memory")
    dev = "cuda"
    stream = workloads.GradientStream(0, D, M, device=dev)
    ctx = tng.Context(D, M, K, tng.CODEC_TERN2, tng.NORM_QUOT, block=128, fuse_mode=tng.FUSE_LSQ)
    hist = []                                         # host copies, oldest first
    for _ in range(K):
        mu = stream.advance()
        ctx.push_reference(mu)
        hist.append(to_np(mu))
    hist = hist[::-1]                                 # newest first, as the fusion numbers them
    out = torch.empty(D, device=dev)
    rng = np.random.default_rng(0)
    rounds = K + 2
    for step in range(rounds):
        stream.advance()
        g = stream.worker_grads()
        if step == rounds - 1:                        # the ring as it stands: the library's own aggregates
            torch.cuda.synchronize()
            hist = [to_np(ctx.history(j)) for j in range(K)]
        ctx.step(g, out)
        torch.cuda.synchronize()
        if step == 0 or step == rounds - 1:
            check_round(ctx, hist, g, out, step, rng)
        del g
    ctx.close()


def test_maximum_vector_length():
    """d = TNG_MAX_COORDS = 2^31 coordinates (8 GiB per vector), one worker, delayed-gradient
    reference: every index computation at the top of its range.  Windows at the far end of the
    vector are checked bit for bit against the oracle (which sees the coordinate offset)."""
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * (1 << 30):
        pytest.skip("needs about 40 GiB of free device memory")
    d = 1 << 31
    dev = "cuda"
    gen = torch.Generator(device=dev)
    gen.manual_seed(11)
    h = torch.empty(d, device=dev).normal_(generator=gen)
    ctx = tng.Context(d, 1, 1, tng.CODEC_TERN2, tng.NORM_DIFF, block=128, seed_lo=9)
    ctx.push_reference(h)
    del h
    g = torch.empty((1, d), device=dev).normal_(generator=gen)
    ctx.step(g)                                          # the aggregate goes to the ring only
    torch.cuda.synchronize()
    st = ctx.stats()
    assert st.pipeline_error == 0 and st.nonfinite_scales == 0 and st.rounds == 1
    codes, scales = ctx.wire()
    newest = ctx.history(0)
    with pytest.raises(tng.TngError):
        tng.Context(d + 1, 1, 1, tng.CODEC_TERN2, tng.NORM_DIFF)
    # the reference of the round was the pushed vector; it has been overwritten by the aggregate
    # (K = 1), so regenerate it
    gen.manual_seed(11)
    h = torch.empty(d, device=dev).normal_(generator=gen)
    for i0, n in [(0, 1024), (d - 2048, 2048), ((1 << 30) - 512, 1024), (d - (1 << 20), 1024)]:
        sl = slice(i0, i0 + n)
        ref = to_np(h[sl])
        wc, ws = oracle.encode(to_np(g[:, sl]), ref, tng.NORM_DIFF, tng.CODEC_TERN2, B=128, seed=(9, 0), t=0, coord_offset=i0)
        t0, t1 = i0 // 128, (i0 + n) // 128
        assert np.array_equal(to_np(codes[:, t0 * 8:t1 * 8]).view(np.uint32), wc), f"codes differ in window {i0}"
        assert np.array_equal(to_np(scales[:, t0:t1]).view(np.uint32), ws.view(np.uint32))
        want = oracle.decode_aggregate(wc, ws, n, ref, tng.NORM_DIFF, tng.CODEC_TERN2, B=128)
        assert np.array_equal(to_np(newest[sl]).view(np.uint32), want.view(np.uint32)), f"aggregate differs in window {i0}"
    ctx.close()
