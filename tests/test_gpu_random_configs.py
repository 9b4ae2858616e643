"""GPU parity on randomly drawn configurations: vector lengths around tile, chunk and block
boundaries, worker counts on both sides of a decode round (32 / b workers) and of a pipeline fill
(8 rows), every codec, normalisation, scale kind and block size, with and without a refresh cadence.
Whole rounds against the oracle, bit for bit, with the fusion modes whose reference involves no
statistics (delayed gradient, window average); the draws are fixed by the seed."""
import numpy as np
import pytest
import torch

from gpu_util import codes_np, drifting_grads, make_ctx, make_oracle, round_up4, same_bits, same_values, to_np
from paper_1901_08227_b200 import tng


def draw(seed):
    rng = np.random.default_rng(1000 + seed)
    kind = rng.integers(0, 4)
    if kind == 0:
        d = int(rng.integers(1, 700))
    elif kind == 1:
        d = int(128 * rng.integers(1, 60) + rng.choice([-1, 0, 1, 3, 64, 127]))
    elif kind == 2:
        d = int(2048 * rng.integers(8, 14) + rng.choice([-129, -1, 0, 1, 128, 130, 2047]))   # staged kernels + tails
    else:
        d = int(rng.integers(700, 40000))
    d = max(d, 1)
    M = int(rng.choice([1, 2, 3, 5, 7, 8, 9, 12, 16, 17, 33, 64], p=[.1, .1, .1, .1, .1, .15, .1, .05, .05, .05, .05, .05]))
    K = int(rng.integers(1, 6))
    codec = int(rng.choice([tng.CODEC_SIGN1, tng.CODEC_TERN2, tng.CODEC_QSGD4]))
    norm = int(rng.choice([tng.NORM_NONE, tng.NORM_DIFF, tng.NORM_QUOT, tng.NORM_COMB, tng.NORM_MEAN]))
    block = int(rng.choice([0, 128, 128, 128, 256, 384, 1024]))
    mode = int(rng.choice([tng.FUSE_LAST, tng.FUSE_MEAN]))
    opts = dict(block=block, fuse_mode=mode, seed_lo=int(rng.integers(0, 2 ** 31)), seed_hi=int(rng.integers(0, 2 ** 31)),
                qsgd_levels=int(rng.integers(1, 8)), scale_kind=int(rng.integers(0, 2)), ref_every=int(rng.choice([1, 1, 2, 3])))
    return d, M, K, codec, norm, opts


def draw_long_blocks(seed):
    """scale blocks of 2 .. 16 tiles in vectors of at least 8 chunks: the one-pass staged kernel plus its tail"""
    rng = np.random.default_rng(9000 + seed)
    d = int(2048 * rng.integers(8, 20) + rng.choice([0, 1, 127, 128, 129, 255, 256, 1023, 1024, 1500, 2047]))
    M = int(rng.choice([1, 2, 5, 8, 9, 16, 17, 64]))
    K = int(rng.integers(1, 5))
    codec = int(rng.choice([tng.CODEC_SIGN1, tng.CODEC_TERN2, tng.CODEC_QSGD4]))
    norm = int(rng.choice([tng.NORM_NONE, tng.NORM_DIFF, tng.NORM_QUOT, tng.NORM_COMB, tng.NORM_MEAN]))
    opts = dict(block=int(rng.choice([256, 512, 1024, 2048])), fuse_mode=int(rng.choice([tng.FUSE_LAST, tng.FUSE_MEAN])),
                seed_lo=int(rng.integers(0, 2 ** 31)), seed_hi=int(rng.integers(0, 2 ** 31)),
                qsgd_levels=int(rng.integers(1, 8)), scale_kind=int(rng.integers(0, 2)), ref_every=int(rng.choice([1, 1, 2])))
    return d, M, K, codec, norm, opts


@pytest.mark.gpu
@pytest.mark.parametrize("seed", range(160))
def test_random_configuration_rounds_are_bit_exact(seed):
    d, M, K, codec, norm, opts = draw(seed) if seed < 120 else draw_long_blocks(seed)
    ctx = make_ctx(d, M, K, codec, norm, **opts)
    orc = make_oracle(d, M, K, codec, norm, **opts)
    out = torch.empty(d, device="cuda")
    what = f"d={d} M={M} K={K} codec={codec} norm={norm} {opts}"
    for t, g in enumerate(drifting_grads(seed, K + 3, M, d, "cuda", ld=round_up4(d) + 4 * (seed % 3))):
        if norm == tng.NORM_MEAN:
            g += 0.25 * (1 + seed % 5)
        ctx.step(g, out)
        want = orc.step(to_np(g))
        codes, scales = ctx.wire()
        assert np.array_equal(codes_np(codes), orc.codes()), f"codes differ at round {t}: {what}"
        assert same_values(to_np(scales), orc.scales()), f"scales differ at round {t}: {what}"
        if norm == tng.NORM_MEAN:
            assert same_bits(to_np(ctx.wire_means()), orc.means()), f"means differ at round {t}: {what}"
        assert same_values(to_np(out), want), f"aggregate differs at round {t}: {what}"
    st = ctx.stats()
    assert st.pipeline_error == 0 and st.rounds == K + 3, what


def draw_fusion(seed):
    rng = np.random.default_rng(5000 + seed)
    k = int(rng.integers(1, 17))                                  # 9..16 take the cross-block statistics kernel
    M = int(rng.choice([1, 2, 3, 5, 8, 9, 16, 24, 64]))
    d = int(rng.choice([rng.integers(1, 3000), 1024 * rng.integers(16, 40) + rng.choice([-1, 0, 1, 515]), rng.integers(3000, 60000)]))
    mode = int(rng.choice([tng.FUSE_LSQ, tng.FUSE_HINDSIGHT]))
    return k, M, d, mode


@pytest.mark.gpu
@pytest.mark.parametrize("seed", range(40))
def test_random_fusion_statistics_and_coefficients(seed):
    """Gram, right-hand side, coefficients and fused reference of randomly drawn histories against
    the oracle, within the tolerances of the fusion tests (1e-10 on the fp64 Gram, 1e-5 on alpha
    and the reference)."""
    import oracle
    from gpu_util import rel_l2
    from paper_1901_08227_b200 import workloads
    k, M, d, mode = draw_fusion(seed)
    ctx = make_ctx(d, M, k, tng.CODEC_TERN2, tng.NORM_DIFF, fuse_mode=mode)
    orc = make_oracle(d, M, k, tng.CODEC_TERN2, tng.NORM_DIFF, fuse_mode=mode)
    traj = workloads.AR1Trajectory(seed, d, device="cuda", rho=0.5)   # weakly correlated: a well-conditioned Gram
    for _ in range(k):
        h = traj.advance().contiguous()
        ctx.push_reference(h)
        orc.push_reference(to_np(h))
    g = traj.worker_grads(M, 0.5, ld=round_up4(d) + 4)
    ctx.fuse(g)
    orc.fuse(to_np(g))
    st = ctx.stats()
    what = f"k={k} M={M} d={d} mode={mode}"
    assert st.k == k and st.solver_fallback == orc.fallback, what
    if orc.fallback:
        return
    G = np.array(st.gram[:]).reshape(16, 16)[:k, :k]
    oG, oc, ogg = orc.gram()
    assert rel_l2(G, oG) < 1e-10, what
    if mode == tng.FUSE_LSQ:
        assert rel_l2(np.array(st.rhs[:k]), oc) < 1e-6 and st.grad_sq == pytest.approx(ogg, rel=1e-6), what
    alpha = np.array(st.alpha[:k])
    assert np.allclose(alpha, orc.alpha().astype(np.float64)[:k], rtol=0, atol=1e-5 * max(1.0, np.abs(alpha).max())), what
    assert rel_l2(to_np(ctx.reference()), orc.ref()) < 1e-5 or not orc.ref().any(), what
