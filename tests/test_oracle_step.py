"""Pins for the oracle's state machine (Algorithm 1): the ring of past aggregates,
the fusion modes, and that a round is the composition of the pinned stages."""
import numpy as np
import pytest

import oracle
from oracle import (CODEC_QSGD4, CODEC_SIGN1, CODEC_TERN2, FUSE_HINDSIGHT, FUSE_LAST, FUSE_LSQ, FUSE_MEAN, NORM_DIFF,
                    NORM_NONE, NORM_QUOT)


def drifting_grads(rng, steps, M, d, noise=0.3):
    mu = rng.standard_normal(d)
    for _ in range(steps):
        mu = 0.95 * mu + 0.1 * rng.standard_normal(d)
        yield (mu[None] + noise * rng.standard_normal((M, d))).astype(np.float32)


def test_first_round_is_plain_compression():
    # Algorithm 1 starts from reference = zeros
    rng = np.random.default_rng(0)
    g = rng.standard_normal((4, 1000)).astype(np.float32)
    st = oracle.State(1000, 4, 3, CODEC_TERN2, NORM_DIFF, block=0, seed_lo=5)
    out = st.step(g)
    codes, sc = oracle.encode(g, None, NORM_NONE, CODEC_TERN2, B=0, seed=(5, 0), t=0)
    assert np.array_equal(st.codes(), codes) and np.array_equal(st.scales(), sc)
    assert np.array_equal(out, oracle.decode_aggregate(codes, sc, 1000, None, NORM_NONE, CODEC_TERN2, B=0))
    assert st.k == 1 and st.t == 1 and np.array_equal(st.history(0), out)


def test_delayed_gradient_reference_K1():
    # reference of round t = averaged decoded TNG of round t-1 (Section 4.2 protocol)
    rng = np.random.default_rng(1)
    st = oracle.State(300, 2, 1, CODEC_TERN2, NORM_DIFF, block=128)
    prev = None
    for t, g in enumerate(drifting_grads(rng, 4, 2, 300)):
        st.fuse(g)
        if prev is None:
            assert not st.ref().any()
        else:
            assert np.array_equal(st.ref(), prev)
        st.encode(g)
        codes, sc = oracle.encode(g, prev, NORM_DIFF, CODEC_TERN2, B=128, t=t)
        assert np.array_equal(st.codes(), codes)
        prev = st.decode_push()
        assert np.array_equal(prev, oracle.decode_aggregate(codes, sc, 300, st.ref(), NORM_DIFF, CODEC_TERN2, B=128))


def test_ring_keeps_the_last_K_aggregates_newest_first():
    st = oracle.State(8, 1, 3, CODEC_TERN2, NORM_DIFF, fuse_mode=FUSE_MEAN)
    vecs = [np.full(8, float(i + 1), dtype=np.float32) for i in range(5)]
    for i, v in enumerate(vecs):
        st.push_reference(v)
        assert st.k == min(i + 1, 3)
        for j in range(st.k):
            assert np.array_equal(st.history(j), vecs[i - j])
    st.fuse(np.zeros((1, 8), dtype=np.float32))
    assert np.array_equal(st.ref(), np.full(8, 4.0, dtype=np.float32))   # mean of 3, 4, 5


@pytest.mark.parametrize("mode", [FUSE_LSQ, FUSE_HINDSIGHT, FUSE_MEAN, FUSE_LAST])
@pytest.mark.parametrize("norm,codec", [(NORM_DIFF, CODEC_TERN2), (NORM_QUOT, CODEC_SIGN1), (NORM_DIFF, CODEC_QSGD4)])
def test_round_is_the_composition_of_the_stages(mode, norm, codec):
    rng = np.random.default_rng(2)
    d, M, K = 700, 3, 4
    st = oracle.State(d, M, K, codec, norm, block=256, fuse_mode=mode, seed_lo=1, seed_hi=2, qsgd_levels=4)
    hist = []
    for t, g in enumerate(drifting_grads(rng, 6, M, d)):
        out = st.step(g)
        if not hist:
            ref = np.zeros(d, dtype=np.float32)
        elif mode == FUSE_LAST:
            ref = hist[0]
        elif mode == FUSE_MEAN:
            ref = oracle.combine(hist, np.full(len(hist), np.float32(1.0) / np.float32(len(hist)), dtype=np.float32))
        else:
            G, c, _ = oracle.fuse_stats(hist, g)
            a32 = oracle.fuse_solve(G, c, 1e-6)[1] if mode == FUSE_LSQ else oracle.fuse_solve_hindsight(G, 1e-6)[1]
            assert np.array_equal(st.alpha()[: len(hist)], a32)
            ref = oracle.combine(hist, a32)
        assert np.array_equal(st.ref(), ref)
        codes, sc = oracle.encode(g, ref, norm, codec, B=256, s=4, seed=(1, 2), t=t)
        assert np.array_equal(st.codes(), codes) and np.array_equal(st.scales(), sc)
        assert np.array_equal(out, oracle.decode_aggregate(codes, sc, d, ref, norm, codec, B=256, s=4))
        hist = [out] + hist[: K - 1]


def test_trajectory_reference_reduces_the_coding_error():
    # the point of the method: ||g - ref||^2 <= C_nz ||g||^2 with C_nz < 1 makes the
    # decoded aggregate closer to the true mean than plain compression of g
    rng = np.random.default_rng(3)
    d, M = 2048, 4
    tng = oracle.State(d, M, 4, CODEC_TERN2, NORM_DIFF, block=128)
    plain = oracle.State(d, M, 1, CODEC_TERN2, NORM_NONE, block=128)
    err_t = err_p = 0.0
    cnz = []
    for t, g in enumerate(drifting_grads(rng, 12, M, d, noise=0.1)):
        gbar = g.astype(np.float64).mean(0)
        tng.fuse(g)
        if t >= 4:
            cnz.append(oracle.cnz(g, tng.ref()))
        tng.encode(g)
        ot = tng.decode_push()
        op = plain.step(g)
        if t >= 4:
            err_t += ((ot - gbar) ** 2).sum()
            err_p += ((op - gbar) ** 2).sum()
    assert max(cnz) < 0.5
    assert err_t < 0.5 * err_p


def test_options_are_validated():
    with pytest.raises(ValueError):
        oracle.State(100, 1, 1, CODEC_TERN2, NORM_DIFF, block=100)
    with pytest.raises(ValueError):
        oracle.State(100, 1, 1, CODEC_QSGD4, NORM_DIFF, qsgd_levels=8)
    with pytest.raises(ValueError):
        oracle.State(100, 1, 17, CODEC_TERN2, NORM_DIFF)
    with pytest.raises(ValueError):
        oracle.State(100, 1, 1, 3, NORM_DIFF)


def test_reference_refresh_cadence_keeps_the_reference_between_refreshes():
    # Sec. 3.1 (last paragraph) / Sec. 4.1: the reference may be refreshed only every tau rounds.
    # With tau = 3 and the delayed-gradient reference, rounds 3..5 all use the aggregate of round 2.
    d, M, K, tau = 300, 3, 2, 3
    rng = np.random.default_rng(2)
    st = oracle.State(d, M, K, oracle.CODEC_TERN2, oracle.NORM_DIFF, fuse_mode=oracle.FUSE_LAST, ref_every=tau, seed_lo=4)
    every = oracle.State(d, M, K, oracle.CODEC_TERN2, oracle.NORM_DIFF, fuse_mode=oracle.FUSE_LAST, ref_every=1, seed_lo=4)
    plain = oracle.State(d, M, K, oracle.CODEC_TERN2, oracle.NORM_DIFF, fuse_mode=oracle.FUSE_LAST, seed_lo=4)
    outs, refs = [], []
    for t in range(8):
        g = rng.standard_normal((M, d)).astype(np.float32)
        outs.append(st.step(g))
        refs.append(st.ref())
        assert np.array_equal(every.step(g), plain.step(g))          # tau = 1 is the default behaviour
    assert not refs[0].any() and not refs[1].any() and not refs[2].any()   # empty ring at the first refresh
    for t in (3, 4, 5):
        assert np.array_equal(refs[t], outs[2])                      # refreshed at t = 3 from the newest aggregate
    for t in (6, 7):
        assert np.array_equal(refs[t], outs[5])
    assert st.k == K and st.t == 8                                   # the ring still took every aggregate
    assert np.array_equal(st.history(0), outs[7]) and np.array_equal(st.history(1), outs[6])
