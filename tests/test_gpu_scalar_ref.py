"""GPU parity of the scalar reference (Section 3.1: reference = mean(g) ones(D), one extra scalar
per worker).  The workers' means (a fixed fp32 tree, so bit for bit), the wire and the aggregate
against the oracle: whole rounds over tile, block and per-vector scales, ragged lengths and
lengths that span several levels of the tree; the stage calls; the workers spread over ranks."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import codes_np, drifting_grads, make_ctx, make_oracle, round_up4, same_bits, same_values, to_np
from paper_1901_08227_b200 import tng

pytestmark = pytest.mark.gpu


def shifted_grads(seed, steps, M, d, ld=None):
    """drifting gradients whose rows have clearly different, non-zero means"""
    shift = torch.linspace(-1.5, 2.5, M, device="cuda")[:, None]
    for g in drifting_grads(seed, steps, M, d, "cuda", ld=ld):
        g += shift
        yield g


@pytest.mark.parametrize("codec,B,d,M", [
    (tng.CODEC_TERN2, 128, 1, 1), (tng.CODEC_TERN2, 128, 100, 3), (tng.CODEC_TERN2, 128, 128 * 9 + 40, 4),
    (tng.CODEC_SIGN1, 128, 2048 * 9 + 128 * 3 + 8, 5), (tng.CODEC_QSGD4, 256, 3000, 4), (tng.CODEC_TERN2, 0, 1000, 4),
    (tng.CODEC_QSGD4, 0, 128 * 1024 + 77, 2),            # more than 1024 tiles: two levels of the tree of the mean
    (tng.CODEC_TERN2, 128, 128 * 1024 * 3 + 128 * 5 + 1, 9), (tng.CODEC_SIGN1, 1024, 128 * 2049, 2)])
def test_rounds_with_the_scalar_reference_are_bit_exact(codec, B, d, M):
    K, steps = 2, 4
    opts = dict(block=B, seed_lo=4, seed_hi=1, qsgd_levels=4)
    ctx = make_ctx(d, M, K, codec, tng.NORM_MEAN, **opts)
    orc = make_oracle(d, M, K, codec, tng.NORM_MEAN, **opts)
    out = torch.empty(d, device="cuda")
    for t, g in enumerate(shifted_grads(21, steps, M, d, ld=round_up4(d) + 8)):
        ctx.step(g, out)
        want = orc.step(to_np(g))
        codes, scales = ctx.wire()
        assert same_bits(to_np(ctx.wire_means()), orc.means()), f"means differ at round {t}"
        assert np.array_equal(codes_np(codes), orc.codes()), f"codes differ at round {t}"
        assert same_values(to_np(scales), orc.scales())
        assert same_values(to_np(out), want), f"aggregate differs at round {t}"
        assert same_values(to_np(ctx.history(0)), want)
    st = ctx.stats()
    assert st.rounds == steps and st.k == K and st.pipeline_error == 0 and st.nonfinite_scales == 0


def test_l2_scale_with_the_scalar_reference():
    d, M = 128 * 40 + 9, 3
    opts = dict(block=512, scale_kind=1, seed_lo=2)
    ctx = make_ctx(d, M, 1, tng.CODEC_QSGD4, tng.NORM_MEAN, **opts)
    orc = make_oracle(d, M, 1, tng.CODEC_QSGD4, tng.NORM_MEAN, **opts)
    out = torch.empty(d, device="cuda")
    for g in shifted_grads(3, 3, M, d):
        ctx.step(g, out)
        want = orc.step(to_np(g))
        assert np.array_equal(codes_np(ctx.wire()[0]), orc.codes())
        assert same_values(to_np(out), want)


def test_stage_calls_with_the_scalar_reference_need_no_fusion():
    d, M = 2048 * 8 + 300, 4
    ctx = make_ctx(d, M, 2, tng.CODEC_TERN2, tng.NORM_MEAN, seed_lo=9)
    g = next(shifted_grads(5, 1, M, d))
    gn = to_np(g)
    ctx.encode(g, step=7)
    mu = oracle.row_means(gn)
    assert same_bits(to_np(ctx.wire_means()), mu)
    wc, ws = oracle.encode(gn, None, tng.NORM_MEAN, tng.CODEC_TERN2, B=128, seed=(9, 0), t=7, means=mu)
    codes, scales = ctx.wire()
    assert np.array_equal(codes_np(codes), wc) and same_values(to_np(scales), ws)
    out = torch.empty(d, device="cuda")
    ctx.decode_aggregate(out)
    want = oracle.decode_aggregate(wc, ws, d, None, tng.NORM_MEAN, tng.CODEC_TERN2, B=128, means=mu)
    assert same_values(to_np(out), want)
    assert ctx.stats().rounds == 0                           # the stage calls do not advance the round


def test_constant_rows_send_zero_codes_and_come_back_exactly():
    d, M = 4096, 4
    cs = torch.tensor([0.5, -1.25, 3.0, 0.0], device="cuda")
    g = cs[:, None].expand(M, d).contiguous()
    ctx = make_ctx(d, M, 1, tng.CODEC_TERN2, tng.NORM_MEAN)
    out = torch.empty(d, device="cuda")
    ctx.step(g, out)
    codes, scales = ctx.wire()
    assert not bool(codes.any()) and not bool(scales.any())
    assert torch.equal(ctx.wire_means(), cs)
    assert torch.equal(out, torch.full((d,), 2.25 / 4, device="cuda"))


def test_a_non_finite_gradient_is_reported():
    d, M = 128 * 20, 2
    ctx = make_ctx(d, M, 1, tng.CODEC_TERN2, tng.NORM_MEAN)
    g = torch.randn(M, d, device="cuda")
    g[1, 777] = float("inf")
    ctx.step(g)
    with pytest.raises(tng.TngError) as e:
        ctx.stats(raise_on_nonfinite=True)
    assert e.value.status == tng.ERR_NONFINITE
    assert ctx.stats().nonfinite_scales >= 1


@pytest.mark.parametrize("P", [2, 4])
def test_workers_spread_over_ranks_with_the_scalar_reference(P):
    """Ranks emulated as contexts in one process; the all-gather done by hand, scalars included."""
    d, M, K, steps = 2048 * 9 + 128 * 3 + 8, 8, 2, 3
    opts = dict(block=128, seed_lo=6)
    ranks = [make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_MEAN, **opts) for _ in range(P)]
    orc = make_oracle(d, M, K, tng.CODEC_TERN2, tng.NORM_MEAN, **opts)
    per = M // P
    outs = [torch.empty(d, device="cuda") for _ in range(P)]
    for t, g in enumerate(shifted_grads(8, steps, M, d)):
        for p, c in enumerate(ranks):
            c.encode_local(g[p * per:(p + 1) * per], p * per, t)
        blocks = [(c.wire_views()[0][p * per:(p + 1) * per].clone(), c.wire_views()[1][p * per:(p + 1) * per].clone(),
                   c.wire_means_view()[p * per:(p + 1) * per].clone()) for p, c in enumerate(ranks)]
        for c in ranks:
            codes, scales = c.wire_views()
            means = c.wire_means_view()
            for p, (bc, bs, bm) in enumerate(blocks):
                codes[p * per:(p + 1) * per].copy_(bc)
                scales[p * per:(p + 1) * per].copy_(bs)
                means[p * per:(p + 1) * per].copy_(bm)
        for c, o in zip(ranks, outs):
            c.decode_commit(o)
        want = orc.step(to_np(g))
        for o in outs:
            assert same_values(to_np(o), want)
        assert np.array_equal(codes_np(ranks[-1].wire()[0]), orc.codes())
        assert same_bits(to_np(ranks[0].wire_means()), orc.means())
