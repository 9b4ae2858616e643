"""Pins for the oracle's scalar reference (Section 3.1: the reference mean(g) ones(D), whose
only cost is one scalar per worker).

The mean is pinned by exact integer arithmetic, by cases whose result depends on the order
of the additions, and by the error bound of pairwise summation; the mode by its reductions
to the plain and the difference forms, by the variance inequality the paper quotes for it,
and by unbiasedness of the decoded aggregate.
"""
import math

import numpy as np
import pytest

import oracle
from oracle import CODEC_QSGD4, CODEC_SIGN1, CODEC_TERN2, NORM_DIFF, NORM_MEAN, NORM_NONE


# ------------------------------------------------------------------ the mean itself
@pytest.mark.parametrize("d", [1, 2, 3, 127, 128, 129, 1000, 4096, 5001])
def test_mean_is_exact_on_small_integers(d):
    """Every partial sum of small integers is exact in fp32, whatever the order, so the tree
    sum is the integer sum; a dropped element or a padding mistake changes it."""
    rng = np.random.default_rng(d)
    g = rng.integers(-64, 65, size=(3, d)).astype(np.float32)
    want = np.array([np.float32(np.float32(int(row.astype(np.int64).sum())) / np.float32(d)) for row in g])
    assert np.array_equal(oracle.row_means(g), want)


def test_mean_takes_adjacent_pairs():
    big = np.float32(2.0 ** 24)
    # (2^24 + 1) + (1 - 2^24): the left pair rounds to 2^24, the right one is exact -> 1.
    # Left to right the sum is 0.
    a = np.array([[big, 1.0, 1.0, -big]], dtype=np.float32)
    assert oracle.row_means(a)[0] == np.float32(0.25)
    # (2^24 - 2^24) + (1 + 1) = 2.  Pairing element i with i + n/2 gives 1.
    b = np.array([[big, -big, 1.0, 1.0]], dtype=np.float32)
    assert oracle.row_means(b)[0] == np.float32(0.5)
    # three elements: (a + b) + (c + 0), divided by 3
    c = np.array([[big, 1.0, 1.0]], dtype=np.float32)
    assert oracle.row_means(c)[0] == np.float32(np.float32(big + np.float32(1.0)) / np.float32(3.0))
    # eight elements, two levels above the pairs
    e = np.array([[big, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, -big]], dtype=np.float32)
    # pairs: 2^24, 2, 2, -(2^24 - 1); then 2^24 + 2, 3 - 2^24; total 5
    assert oracle.row_means(e)[0] == np.float32(5.0 / 8.0)


def test_mean_is_within_the_pairwise_summation_bound():
    rng = np.random.default_rng(1)
    for d in (777, 5000, 70001):
        g = (rng.standard_normal((2, d)) * np.exp(rng.uniform(-3, 3, size=(2, d)))).astype(np.float32)
        got = oracle.row_means(g)
        for m in range(2):
            exact = math.fsum(float(x) for x in g[m]) / d
            depth = math.ceil(math.log2(d)) + 1                  # tree levels + the division
            bound = depth * 2.0 ** -24 * math.fsum(abs(float(x)) for x in g[m]) / d * 1.01
            assert abs(float(got[m]) - exact) <= bound


def test_mean_of_means_is_the_sequential_fp32_average():
    mu = np.array([1.0, 2.0, 4.0], dtype=np.float32)
    assert oracle.mean_of_means(mu) == np.float32(np.float32(7.0) / np.float32(3.0))
    big = np.float32(2.0 ** 24)
    # ((2^24 + 1) + 1) - 2^24 = 0 taken left to right (a pairwise sum would give 1/4... of 1)
    assert oracle.mean_of_means(np.array([big, 1.0, 1.0, -big], dtype=np.float32)) == np.float32(0.0)
    assert oracle.mean_of_means(np.array([3.5], dtype=np.float32)) == np.float32(3.5)


def test_subtracting_the_mean_never_increases_the_energy():
    """The inequality the paper quotes for this reference: E||a - E a||^2 <= E||a||^2."""
    rng = np.random.default_rng(2)
    for shift in (0.0, 0.3, -5.0):
        g = (rng.standard_normal((4, 3000)) + shift).astype(np.float32)
        mu = oracle.row_means(g).astype(np.float64)
        centred = ((g.astype(np.float64) - mu[:, None]) ** 2).sum(axis=1)
        plain = (g.astype(np.float64) ** 2).sum(axis=1)
        assert np.all(centred <= plain * (1 + 1e-6))
        if shift != 0.0:
            assert np.all(centred < 0.95 * plain)


# ------------------------------------------------------------------ the mode
@pytest.mark.parametrize("codec", [CODEC_SIGN1, CODEC_TERN2, CODEC_QSGD4])
def test_zero_mean_rows_reduce_to_plain_compression(codec):
    rng = np.random.default_rng(3)
    half = rng.standard_normal((3, 333)).astype(np.float32)
    g = np.empty((3, 666), dtype=np.float32)
    g[:, 0::2] = half                                            # adjacent pairs cancel exactly
    g[:, 1::2] = -half
    assert np.array_equal(oracle.row_means(g), np.zeros(3, dtype=np.float32))
    for B in (0, 128, 256):
        c0, s0 = oracle.encode(g, None, NORM_NONE, codec, B=B, t=4, seed=(1, 2))
        c1, s1 = oracle.encode(g, None, NORM_MEAN, codec, B=B, t=4, seed=(1, 2))
        assert np.array_equal(c0, c1) and np.array_equal(s0, s1)
        o0 = oracle.decode_aggregate(c0, s0, 666, None, NORM_NONE, codec, B=B)
        o1 = oracle.decode_aggregate(c1, s1, 666, None, NORM_MEAN, codec, B=B, means=np.zeros(3, dtype=np.float32))
        assert np.array_equal(o0, o1)


def test_constant_rows_cost_nothing_but_their_scalar():
    d, M = 512, 4
    cs = np.array([0.5, -1.25, 3.0, 0.0], dtype=np.float32)
    g = np.repeat(cs[:, None], d, axis=1)
    mu = oracle.row_means(g)
    assert np.array_equal(mu, cs)
    codes, scales = oracle.encode(g, None, NORM_MEAN, CODEC_TERN2, B=128, means=mu)
    assert not codes.any() and not scales.any()
    out = oracle.decode_aggregate(codes, scales, d, None, NORM_MEAN, CODEC_TERN2, B=128, means=mu)
    assert np.array_equal(out, np.full(d, np.float32(2.25 / 4), dtype=np.float32))


@pytest.mark.parametrize("codec", [CODEC_SIGN1, CODEC_TERN2, CODEC_QSGD4])
def test_one_worker_is_the_difference_form_with_a_constant_reference(codec):
    rng = np.random.default_rng(5)
    d = 128 * 5 + 17
    g = (rng.standard_normal((1, d)) + 0.7).astype(np.float32)
    mu = oracle.row_means(g)
    ref = np.full(d, mu[0], dtype=np.float32)
    for B in (0, 128):
        c1, s1 = oracle.encode(g, None, NORM_MEAN, codec, B=B, t=2, seed=(7, 0), means=mu)
        c2, s2 = oracle.encode(g, ref, NORM_DIFF, codec, B=B, t=2, seed=(7, 0))
        assert np.array_equal(c1, c2) and np.array_equal(s1, s2)
        o1 = oracle.decode_aggregate(c1, s1, d, None, NORM_MEAN, codec, B=B, means=mu)
        o2 = oracle.decode_aggregate(c2, s2, d, ref, NORM_DIFF, codec, B=B)
        assert np.array_equal(o1, o2)


def test_each_worker_is_centred_by_its_own_scalar():
    """Workers with different means: every row's codes are those of that row alone."""
    rng = np.random.default_rng(6)
    d, M = 700, 3
    g = (rng.standard_normal((M, d)) + np.array([[2.0], [-1.0], [0.25]])).astype(np.float32)
    mu = oracle.row_means(g)
    codes, scales = oracle.encode(g, None, NORM_MEAN, CODEC_TERN2, B=128, t=1, means=mu)
    for m in range(M):
        ref = np.full(d, mu[m], dtype=np.float32)
        cm, sm = oracle.encode(g, ref, NORM_DIFF, CODEC_TERN2, B=128, t=1)     # all rows against mu[m]
        assert np.array_equal(codes[m], cm[m]) and np.array_equal(scales[m], sm[m])


def test_decoded_aggregate_is_unbiased():
    """Mean over many seeds of the decoded aggregate = the average gradient, within the
    sampling error of the ternary code; leaving the scalars out would shift every element."""
    rng = np.random.default_rng(7)
    d, M, S = 256, 4, 1500
    g = (0.3 * rng.standard_normal((M, d)) + np.array([[1.0], [2.0], [-0.5], [4.0]])).astype(np.float32)
    mu = oracle.row_means(g)
    acc = np.zeros(d)
    for s in range(S):
        codes, scales = oracle.encode(g, None, NORM_MEAN, CODEC_TERN2, B=128, t=s, seed=(s, 3), means=mu)
        acc += oracle.decode_aggregate(codes, scales, d, None, NORM_MEAN, CODEC_TERN2, B=128, means=mu)
    est = acc / S
    want = g.astype(np.float64).mean(axis=0)
    v = g.astype(np.float64) - mu[:, None].astype(np.float64)
    R = np.repeat(np.abs(v).reshape(M, d // 128, 128).max(axis=2), 128, axis=1)
    var = (R * np.abs(v) - v * v).sum(axis=0) / M ** 2           # ternary variance, averaged over workers
    z = np.abs(est - want) / np.sqrt(var / S + 1e-12)
    assert z.max() < 5.5
    assert abs(float(np.mean(est - want))) < 3e-3                # no common shift (the scalars average 1.625)


def test_a_window_with_the_whole_vectors_means_equals_the_window_of_the_whole_encode():
    rng = np.random.default_rng(8)
    d = 128 * 9
    g = (rng.standard_normal((2, d)) + 1.5).astype(np.float32)
    mu = oracle.row_means(g)
    codes, scales = oracle.encode(g, None, NORM_MEAN, CODEC_TERN2, B=128, t=3, means=mu)
    i0, n = 128 * 4, 128 * 3
    wc, ws = oracle.encode(np.ascontiguousarray(g[:, i0:i0 + n]), None, NORM_MEAN, CODEC_TERN2, B=128, t=3,
                           coord_offset=i0, means=mu)
    assert np.array_equal(wc, codes[:, 8 * 4:8 * 7]) and np.array_equal(ws, scales[:, 4:7])


# ------------------------------------------------------------------ the round
def test_round_with_the_scalar_reference_ignores_the_trajectory():
    rng = np.random.default_rng(9)
    d, M, K = 128 * 3 + 40, 3, 2
    outs = []
    for push in (False, True):
        st = oracle.State(d, M, K, CODEC_TERN2, NORM_MEAN, seed_lo=5)
        if push:
            st.push_reference(rng.standard_normal(d).astype(np.float32))
        rng2 = np.random.default_rng(10)
        rounds = []
        for t in range(3):
            g = (rng2.standard_normal((M, d)) + 0.5 * t).astype(np.float32)
            out = st.step(g)
            mu = oracle.row_means(g)
            assert np.array_equal(st.means(), mu)
            codes, scales = oracle.encode(g, None, NORM_MEAN, CODEC_TERN2, B=128, t=t, seed=(5, 0), means=mu)
            assert np.array_equal(st.codes(), codes) and np.array_equal(st.scales(), scales)
            want = oracle.decode_aggregate(codes, scales, d, None, NORM_MEAN, CODEC_TERN2, B=128, means=mu)
            assert np.array_equal(out, want)
            assert np.array_equal(st.history(0), out)            # the aggregate still enters the ring
            rounds.append(out)
        outs.append(rounds)
        st.close()
    for a, b in zip(*outs):
        assert np.array_equal(a, b)
