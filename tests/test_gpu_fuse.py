"""GPU parity of the trajectory fusion (Gram statistics, K x K solve, combine) and of
whole rounds (tng_step) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import same_numbers, codes_np, drifting_grads, make_ctx, make_oracle, rel_l2, same_values, to_np
from paper_1901_08227_b200 import tng, workloads

pytestmark = pytest.mark.gpu

TOL = 1e-5          # relative L2 bound on references, Gram coefficients and aggregates


def gram_of(stats, k):
    G = np.array(stats.gram[:]).reshape(16, 16)[:k, :k]
    return G, np.array(stats.rhs[:k]), stats.grad_sq


@pytest.mark.parametrize("k,M,d", [(1, 1, 5), (2, 4, 1000), (4, 16, 65536 + 3), (8, 8, 128 * 5000 + 77), (11, 3, 40001), (16, 2, 9000)])
@pytest.mark.parametrize("mode", [tng.FUSE_LSQ, tng.FUSE_HINDSIGHT, tng.FUSE_MEAN])
def test_fusion_stage(k, M, d, mode):
    dev = "cuda"
    K = max(k, 1)
    ctx = make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_DIFF, fuse_mode=mode)
    orc = make_oracle(d, M, K, tng.CODEC_TERN2, tng.NORM_DIFF, fuse_mode=mode)
    traj = workloads.AR1Trajectory(k * 31 + M, d, device=dev, rho=0.9)
    for _ in range(k):
        h = traj.advance().contiguous()
        ctx.push_reference(h)
        orc.push_reference(to_np(h))
    g = traj.worker_grads(M, 0.5, ld=(d + 3) // 4 * 4 + 8)
    ctx.fuse(g)
    ref = to_np(ctx.reference())
    st = ctx.stats()
    orc.fuse(to_np(g))
    assert st.k == k and st.solver_fallback == orc.fallback == 0
    alpha = np.array(st.alpha[:k])
    assert np.allclose(alpha, orc.alpha().astype(np.float64)[:k], rtol=0, atol=TOL * max(1.0, np.abs(alpha).max()))
    assert rel_l2(ref, orc.ref()) < TOL
    if mode != tng.FUSE_MEAN:
        G, c, gg = gram_of(st, k)
        oG, oc, ogg = orc.gram()
        assert rel_l2(G, oG) < 1e-10
        if mode == tng.FUSE_LSQ:
            assert rel_l2(c, oc) < 1e-6 and gg == pytest.approx(ogg, rel=1e-6)
            assert st.cnz == pytest.approx(oracle.cnz(to_np(g), orc.ref()), rel=1e-4)
    else:
        assert same_values(ref, orc.ref())        # same fp32 fma chain: bit exact
    for j in range(k):
        assert same_values(to_np(ctx.history(j)), orc.history(j))


def test_rank_deficient_history_falls_back():
    d, M = 3000, 2
    ctx = make_ctx(d, M, 3, tng.CODEC_TERN2, tng.NORM_DIFF, ridge=0.0)
    orc = make_oracle(d, M, 3, tng.CODEC_TERN2, tng.NORM_DIFF, ridge=0.0)
    h = workloads.normal((d,), 1, 0, "cuda")
    for _ in range(3):
        ctx.push_reference(h)
        orc.push_reference(to_np(h))
    g = workloads.random_grads(2, M, d, device="cuda")
    ctx.fuse(g)
    orc.fuse(to_np(g))
    st = ctx.stats()
    assert st.solver_fallback == 1 and orc.fallback == 1
    assert list(st.alpha[:3]) == [1.0, 0.0, 0.0]
    assert same_values(to_np(ctx.reference()), to_np(h))


@pytest.mark.parametrize("mode,K", [(tng.FUSE_LAST, 1), (tng.FUSE_LAST, 3), (tng.FUSE_MEAN, 4)])
@pytest.mark.parametrize("norm,codec,B", [(tng.NORM_DIFF, tng.CODEC_TERN2, 0), (tng.NORM_QUOT, tng.CODEC_TERN2, 128),
                                          (tng.NORM_DIFF, tng.CODEC_QSGD4, 256), (tng.NORM_DIFF, tng.CODEC_SIGN1, 128)])
@pytest.mark.parametrize("d", [128 * 9 + 40, 1024 * 18 + 128 * 7 + 40])
def test_rounds_are_bit_exact_when_the_reference_is(mode, K, norm, codec, B, d):
    # delayed-gradient and window-average references are exact fp32 on both sides,
    # so whole trajectories (codes, scales, aggregates, ring) agree bit for bit
    # (the longer vectors go through the staged kernels, the window average being
    # combined inside the encode pass)
    M, steps = 4, 7
    opts = dict(block=B, fuse_mode=mode, seed_lo=21, seed_hi=4, qsgd_levels=4)
    ctx = make_ctx(d, M, K, codec, norm, **opts)
    orc = make_oracle(d, M, K, codec, norm, **opts)
    out = torch.empty(d, device="cuda")
    for t, g in enumerate(drifting_grads(77, steps, M, d, "cuda", ld=d + 8)):
        ctx.step(g, out)
        codes, scales = ctx.wire()
        want = orc.step(to_np(g))
        assert np.array_equal(codes_np(codes), orc.codes()), f"codes differ at round {t}"
        assert same_values(to_np(scales), orc.scales())
        assert same_values(to_np(out), want)
        assert same_values(to_np(ctx.history(0)), want)
        if not (mode == tng.FUSE_LAST and K == 1):
            # (with K = 1 the delayed-gradient reference aliases the only ring slot, which the
            # round has just overwritten with the new aggregate)
            # The delayed-gradient reference IS the newest ring entry on the GPU (no pass), while the oracle
            # forms fma(1, h, +0): a -0 entry stays -0 on one side and becomes +0 on the other.  Nothing the
            # round computes depends on the sign of a zero reference element (the aggregates above are
            # compared bit for bit), so the reference itself is compared as numbers there.
            same = same_numbers if mode == tng.FUSE_LAST else same_values
            assert same(to_np(ctx.reference()), orc.ref())
    st = ctx.stats()
    assert st.rounds == steps and st.k == min(steps, K) and st.kernel_launches > 0


@pytest.mark.parametrize("mode", [tng.FUSE_LSQ, tng.FUSE_HINDSIGHT])
@pytest.mark.parametrize("norm,codec,B,K", [(tng.NORM_DIFF, tng.CODEC_QSGD4, 256, 4), (tng.NORM_QUOT, tng.CODEC_TERN2, 128, 8),
                                            (tng.NORM_DIFF, tng.CODEC_SIGN1, 128, 3)])
def test_least_squares_rounds_stage_by_stage(mode, norm, codec, B, K):
    # The fused reference is only equal to 1e-5, so each round is checked stage-wise:
    # the GPU fusion against the oracle's within tolerance; then encode and decode on the
    # GPU *given the oracle's reference*, bit for bit; the GPU ring receives the same vector.
    d, M, steps = 128 * 30 + 5, 4, 2 * K + 2
    opts = dict(block=B, fuse_mode=mode, seed_lo=8, qsgd_levels=4)
    ctx = make_ctx(d, M, K, codec, norm, **opts)
    orc = make_oracle(d, M, K, codec, norm, **opts)
    out = torch.empty(d, device="cuda")
    for t, g in enumerate(drifting_grads(5, steps, M, d, "cuda")):
        gn = to_np(g)
        ctx.fuse(g)
        orc.fuse(gn)
        oref = orc.ref()
        assert rel_l2(to_np(ctx.reference()), oref) < TOL or not oref.any()
        ref_dev = torch.from_numpy(oref).cuda()
        ctx.encode(g, ref=ref_dev, step=t)
        orc.encode(gn)
        codes, scales = ctx.wire()
        assert np.array_equal(codes_np(codes), orc.codes()), f"codes differ at round {t}"
        assert same_values(to_np(scales), orc.scales())
        ctx.decode_aggregate(out, ref=ref_dev)
        want = orc.decode_push()
        assert same_values(to_np(out), want)
        ctx.push_reference(out)


@pytest.mark.parametrize("mode", [tng.FUSE_LSQ, tng.FUSE_HINDSIGHT])
@pytest.mark.parametrize("d,M,K", [(128 * 64 + 9, 8, 4), (1024 * 40 + 128 * 3 + 72, 8, 8), (1024 * 21 + 130, 19, 3)])
def test_step_equals_its_own_stages_and_tracks_the_oracle(mode, d, M, K):
    # tng_step must be exactly fuse -> encode(step = round) -> decode -> push on the GPU,
    # and its aggregates must stay within tolerance of the oracle's trajectory except where a
    # last-bit difference of the reference flips a stochastic rounding (rare).
    steps = 10
    opts = dict(block=128, fuse_mode=mode, seed_lo=99)
    a = make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_DIFF, **opts)
    b = make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_DIFF, **opts)
    orc = make_oracle(d, M, K, tng.CODEC_TERN2, tng.NORM_DIFF, **opts)
    out_a = torch.empty(d, device="cuda")
    out_b = torch.empty(d, device="cuda")
    rels = []
    exact_rounds = 0
    for t, g in enumerate(drifting_grads(6, steps, M, d, "cuda")):
        a.step(g, out_a)
        b.fuse(g)
        b.encode(g, step=t)
        b.decode_aggregate(out_b)
        b.push_reference(out_b)
        assert torch.equal(out_a, out_b)
        assert torch.equal(a.wire()[0], b.wire()[0])
        want = orc.step(to_np(g))
        got = to_np(out_a)
        rels.append(rel_l2(got, want))
        if t == 0:
            assert same_values(got, want)            # empty ring: zero reference on both sides
        # Every sum the coefficients depend on is a double sum on both sides, so the fp32 coefficients come
        # out identical (a difference needs alpha to sit within ~1e-13 of a rounding boundary) and with them
        # the reference, the codes and the aggregate: the trajectories agree bit for bit.
        k = min(t, K)
        if np.array_equal(np.array(a.stats().alpha[:k]).astype(np.float32), orc.alpha()[:k]):
            exact_rounds += 1
            assert same_values(got, want), f"round {t}: same coefficients but a different aggregate"
    # were a rounding ever to flip, it would move one coordinate by R/M (about 1e-3 of the norm here) and stay in the ring
    assert max(rels) < 5e-3
    assert np.median(rels) < TOL
    assert exact_rounds == steps, f"only {exact_rounds} of {steps} rounds had identical coefficients"
    assert a.stats().pipeline_error == 0 and b.stats().pipeline_error == 0
