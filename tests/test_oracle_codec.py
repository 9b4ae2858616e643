"""Pins for the oracle's normalise / scale / quantise / pack / decode stages.

Each test compares the oracle with something it does not compute itself: exact
values on grid points, the closed-form mean and variance of each code
(Section 3.2 gives the ternary distribution; the others follow from their
definitions), an independent unpacker of the wire layout, numpy in float64.
"""
import numpy as np
import pytest

import oracle
from oracle import (CODEC_QSGD4, CODEC_SIGN1, CODEC_TERN2, NORM_DIFF, NORM_NONE, NORM_QUOT, SCALE_ABSMAX,
                    SCALE_L2)


def unpack_symbols(codes_m, d, b):
    """Independent reader of the tile-planar layout: tile T owns 4b words; word
    c*b+p, bit j, is bit p of the symbol of coordinate 128T + 4j + c."""
    sym = np.zeros(d, dtype=np.uint32)
    for i in range(d):
        T, within = divmod(i, 128)
        j, c = divmod(within, 4)
        for p in range(b):
            sym[i] |= ((int(codes_m[T * 4 * b + c * b + p]) >> j) & 1) << p
    return sym


def grid_vector(rng, d, R, levels):
    """values in {-R, ..., -R/levels, 0, R/levels, ..., R} with both extremes present"""
    v = (rng.integers(-levels, levels + 1, size=d) * (R / levels)).astype(np.float32)
    v[rng.integers(0, d)] = R
    return v


# ------------------------------------------------------------------ exactness on grid points
@pytest.mark.parametrize("d", [1, 5, 128, 129, 1000])
@pytest.mark.parametrize("R", [1.0, 0.375, 3.0e-5])
def test_ternary_is_exact_on_its_grid(d, R):
    rng = np.random.default_rng(d)
    v = grid_vector(rng, d, np.float32(R), 1)
    for t in range(5):
        codes, scales = oracle.encode(v[None], None, NORM_NONE, CODEC_TERN2, B=0, t=t, seed=(t, 1))
        assert scales[0, 0] == np.float32(R)
        out = oracle.decode_aggregate(codes, scales, d, None, NORM_NONE, CODEC_TERN2, B=0)
        assert np.array_equal(out, v)


def test_sign_is_exact_on_plus_minus_R():
    rng = np.random.default_rng(0)
    v = (rng.choice([-1.0, 1.0], size=777) * 0.8125).astype(np.float32)
    for t in range(5):
        codes, scales = oracle.encode(v[None], None, NORM_NONE, CODEC_SIGN1, B=128, t=t)
        out = oracle.decode_aggregate(codes, scales, 777, None, NORM_NONE, CODEC_SIGN1, B=128)
        assert np.array_equal(out, v)


@pytest.mark.parametrize("s", [1, 2, 4])
def test_qsgd_is_exact_on_its_grid_for_dyadic_scales(s):
    rng = np.random.default_rng(s)
    for R in [1.0, 0.25, 64.0]:
        v = grid_vector(rng, 900, np.float32(R), s)
        codes, scales = oracle.encode(v[None], None, NORM_NONE, CODEC_QSGD4, B=256, s=s, t=3)
        out = oracle.decode_aggregate(codes, scales, 900, None, NORM_NONE, CODEC_QSGD4, B=256, s=s)
        # every block holds +-R with overwhelming probability; compare where it does
        for blk in range(4):
            sl = slice(blk * 256, min(900, (blk + 1) * 256))
            if scales[0, blk] == np.float32(R):
                assert np.array_equal(out[sl], v[sl])


def test_qsgd_one_level_equals_ternary_on_dyadic_inputs():
    rng = np.random.default_rng(5)
    v = (rng.integers(-256, 257, size=1000) / 256.0).astype(np.float32)
    v[17] = 1.0
    ct, st_ = oracle.encode(v[None], None, NORM_NONE, CODEC_TERN2, B=0, t=9, seed=(4, 4))
    cq, sq = oracle.encode(v[None], None, NORM_NONE, CODEC_QSGD4, B=0, s=1, t=9, seed=(4, 4))
    tern = unpack_symbols(ct[0], 1000, 2)
    qs = unpack_symbols(cq[0], 1000, 4)
    assert np.array_equal(tern & 1, qs & 1)
    assert np.array_equal(tern >> 1, qs >> 3)
    assert st_[0, 0] == sq[0, 0] == 1.0


# ------------------------------------------------------------------ wire layout and size
@pytest.mark.parametrize("d", list(range(1, 40)) + [127, 128, 129, 255, 256, 257, 383, 511, 600])
def test_pack_layout_roundtrip(d):
    rng = np.random.default_rng(d)
    # deterministic symbols: ternary on {-1,0,1}, so symbol = (nz, neg) is known without the RNG
    v = rng.integers(-1, 2, size=d).astype(np.float32)
    v[rng.integers(0, d)] = 1.0
    codes, _ = oracle.encode(v[None], None, NORM_NONE, CODEC_TERN2, B=0)
    sym = unpack_symbols(codes[0], d, 2)
    assert np.array_equal(sym & 1, (v != 0).astype(np.uint32))
    assert np.array_equal(sym >> 1, (v < 0).astype(np.uint32))
    # bits of coordinates >= d stay zero
    total = int(sum(bin(int(w)).count("1") for w in codes[0]))
    assert total == int((v != 0).sum() + (v < 0).sum())
    assert codes.shape[1] == -(-d // 128) * 8


def test_qsgd_and_sign_planes():
    v = np.array([1.0, -1.0, 0.5, -0.5, 0.25, -0.75, 0.0] + [0.0] * 130, dtype=np.float32)
    codes, scales = oracle.encode(v[None], None, NORM_NONE, CODEC_QSGD4, B=0, s=4)
    sym = unpack_symbols(codes[0], len(v), 4)
    assert list(sym[:7]) == [4, 8 | 4, 2, 8 | 2, 1, 8 | 3, 0]
    w = np.array([2.0, -2.0] * 70, dtype=np.float32)
    codes, _ = oracle.encode(w[None], None, NORM_NONE, CODEC_SIGN1, B=0)
    assert list(unpack_symbols(codes[0], len(w), 1)) == [1, 0] * 70


def test_dense_ternary_costs_two_bits_per_element():
    # Section 4.1 counts a 16-bit reference round as 8 ternary rounds: 2 bits/element
    for d in [128, 1024, 1 << 20]:
        assert oracle.words_per_worker(d, CODEC_TERN2) * 32 / d == 2.0
    assert oracle.bits_per_coord(1 << 27, 8, CODEC_TERN2, 128) == pytest.approx(2 + 0.25 + 512 / 2 ** 27)
    assert oracle.bits_per_coord(1000, 1, CODEC_TERN2, 0) == pytest.approx(2 + 32 / 1000 + 64 / 1000)


# ------------------------------------------------------------------ unbiasedness and variance
def _moments(v, codec, S, **kw):
    d = len(v)
    acc = np.zeros(d)
    acc2 = np.zeros(d)
    R = None
    for t in range(S):
        codes, scales = oracle.encode(v[None], None, NORM_NONE, codec, t=t, **kw)
        out = oracle.decode_aggregate(codes, scales, d, None, NORM_NONE, codec,
                                      **{k: kw[k] for k in kw if k in ("B", "s")}).astype(np.float64)
        acc += out
        acc2 += out * out
        R = scales
    mean = acc / S
    var = acc2 / S - mean ** 2
    return mean, var, R


def _check_moments(v, mean, var, var_closed, S, R):
    vd = v.astype(np.float64)
    se = np.sqrt(var_closed / S)
    z = np.abs(mean - vd) / np.maximum(se, 1e-30)
    z = np.where(var_closed == 0, 0.0, z)
    assert np.all(np.abs(mean - vd)[var_closed == 0] == 0)
    assert z.max() < 5.5, z.max()                       # per-coordinate CI (E Q[v] = v)
    assert abs(np.mean((mean - vd) / R)) < 5.0 / np.sqrt(S * len(v))   # no common bias
    # variance matches the closed form on average
    assert np.sum(var) == pytest.approx(np.sum(var_closed), rel=0.05)


def test_ternary_unbiased_with_closed_form_variance():
    rng = np.random.default_rng(11)
    d, S = 512, 1500
    v = rng.standard_normal(d).astype(np.float32)
    mean, var, scales = _moments(v, CODEC_TERN2, S, B=0, seed=(1, 2))
    R = float(scales[0, 0])
    assert R == np.abs(v).max()                        # R = max_d |v_d|
    _check_moments(v, mean, var, R * np.abs(v.astype(np.float64)) - v.astype(np.float64) ** 2, S, R)


def test_ternary_nonzero_fraction():
    rng = np.random.default_rng(12)
    v = rng.standard_normal(1 << 14).astype(np.float32)
    codes, scales = oracle.encode(v[None], None, NORM_NONE, CODEC_TERN2, B=0, t=1)
    nz = (unpack_symbols(codes[0], len(v), 2) & 1).mean()
    p = np.abs(v).mean() / scales[0, 0]
    assert abs(nz - p) < 5 * np.sqrt(p * (1 - p) / len(v))


def test_sign_unbiased_with_closed_form_variance():
    rng = np.random.default_rng(13)
    d, S = 384, 2500
    v = rng.uniform(-1, 1, d).astype(np.float32)
    mean, var, scales = _moments(v, CODEC_SIGN1, S, B=128, seed=(3, 4))
    Rv = np.repeat(scales[0].astype(np.float64), 128)[:d]
    _check_moments(v, mean, var, Rv ** 2 - v.astype(np.float64) ** 2, S, Rv)


@pytest.mark.parametrize("s", [2, 4, 7])
def test_qsgd_unbiased_with_closed_form_variance(s):
    rng = np.random.default_rng(14 + s)
    d, S = 256, 1500
    v = rng.standard_normal(d).astype(np.float32)
    mean, var, scales = _moments(v, CODEC_QSGD4, S, B=128, s=s, seed=(5, 6))
    Rv = np.repeat(scales[0].astype(np.float64), 128)[:d]
    a = np.abs(v.astype(np.float64)) / Rv * s
    f = a - np.floor(a)
    _check_moments(v, mean, var, (Rv / s) ** 2 * f * (1 - f), S, Rv)


def test_qsgd_l2_scale_unbiased():
    rng = np.random.default_rng(21)
    d, S = 256, 1500
    v = rng.standard_normal(d).astype(np.float32)
    mean, var, scales = _moments(v, CODEC_QSGD4, S, B=128, s=7, scale_kind=SCALE_L2)
    Rv = np.repeat(scales[0].astype(np.float64), 128)[:d]
    a = np.abs(v.astype(np.float64)) / Rv * 7
    f = a - np.floor(a)
    _check_moments(v, mean, var, (Rv / 7) ** 2 * f * (1 - f), S, Rv)


def test_qsgd_level_never_exceeds_s_when_the_l2_scale_underestimates():
    # The cited s-level quantiser has levels 0..s and nothing above.  With the L2 scale and a block whose
    # squares are subnormal, sqrt(fl(v*v)) < |v|, so |v|/R > 1 and floor(a) + 1 would be s + 1: in the
    # 4-bit symbol that spills into the sign bit.  The level is therefore bounded by s.
    s = 7
    for x in (1e-22, 3e-22, -1e-22, -3e-22):
        v = np.zeros(128, dtype=np.float32)
        v[37] = x
        R = np.sqrt(np.float32(v[37] * v[37]))
        assert R > 0 and abs(np.float32(x)) / R > 1.0          # the premise of the case
        for t in range(200):
            codes, sc = oracle.encode(v[None], None, NORM_NONE, CODEC_QSGD4, B=128, s=s, scale_kind=SCALE_L2, t=t)
            assert sc[0, 0] == R
            sym = unpack_symbols(codes[0], 128, 4)
            assert (sym & 7)[37] <= s
            assert (sym[37] >> 3) == (1 if x < 0 else 0)           # sign bit = (v < 0), not a spilt level bit
            assert (sym & 7)[37] == s                               # a >= s: the top level, always
            assert not np.delete(sym, 37).any()
            out = oracle.decode_aggregate(codes, sc, 128, None, NORM_NONE, CODEC_QSGD4, B=128, s=s)
            assert (out[37] > 0) == (x > 0) and abs(out[37]) == np.float32(np.float32(s) * np.float32(R / np.float32(s)))


def test_qsgd_level_bound_changes_nothing_in_the_normal_range():
    # in the normal range a <= s up to rounding; when a == s exactly, floor(a) = s and frac = 0, so the
    # bound is never active: the symbols equal an independent numpy restatement without it
    rng = np.random.default_rng(77)
    d, s = 512, 7
    v = rng.standard_normal(d).astype(np.float32)
    for kind in (SCALE_ABSMAX, SCALE_L2):
        for t in range(20):
            codes, sc = oracle.encode(v[None], None, NORM_NONE, CODEC_QSGD4, B=128, s=s, scale_kind=kind, t=t, seed=(3, 9))
            sym = unpack_symbols(codes[0], d, 4)
            R = np.repeat(sc[0], 128)[:d]
            a = (np.abs(v) / R).astype(np.float32) * np.float32(s)
            l = np.floor(a)
            f = (a - l).astype(np.float32)
            u = np.array([oracle.coord_uniform(3, 9, i, 0, t) for i in range(d)], dtype=np.float32)
            L = l.astype(np.int64) + (u < f)
            assert L.max() <= s
            assert np.array_equal(sym & 7, L.astype(np.uint32))
            assert np.array_equal(sym >> 3, ((L > 0) & (v < 0)).astype(np.uint32))


# ------------------------------------------------------------------ scales
def test_absmax_scale_per_block_and_per_vector():
    rng = np.random.default_rng(3)
    g = rng.standard_normal((3, 1000)).astype(np.float32)
    _, sc = oracle.encode(g, None, NORM_NONE, CODEC_TERN2, B=256)
    want = np.stack([[np.abs(g[m, b * 256:(b + 1) * 256]).max() for b in range(4)] for m in range(3)])
    assert np.array_equal(sc, want)
    _, sc = oracle.encode(g, None, NORM_NONE, CODEC_TERN2, B=0)
    assert np.array_equal(sc[:, 0], np.abs(g).max(axis=1))


def test_l2_scale_value_and_tree_shape():
    rng = np.random.default_rng(4)
    g = rng.standard_normal((2, 640)).astype(np.float32)
    _, sc = oracle.encode(g, None, NORM_NONE, CODEC_QSGD4, B=128, scale_kind=SCALE_L2)
    want = np.stack([[np.linalg.norm(g[m, b * 128:(b + 1) * 128].astype(np.float64)) for b in range(5)]
                     for m in range(2)])
    assert np.allclose(sc, want, rtol=2e-6)
    # exact sums of dyadic squares
    v = np.array([3.0, 4.0] + [0.0] * 126, dtype=np.float32)
    _, sc = oracle.encode(v[None], None, NORM_NONE, CODEC_QSGD4, B=128, scale_kind=SCALE_L2)
    assert sc[0, 0] == 5.0
    # adjacent-pairwise tree: (1 + e) + (e + e) keeps 2e where a left-to-right sum loses all three
    e = 2.0 ** -12                                      # e^2 = 2^-24 = half an ulp of 1
    v = np.array([1.0, e, e, e] + [0.0] * 124, dtype=np.float32)
    _, sc = oracle.encode(v[None], None, NORM_NONE, CODEC_QSGD4, B=128, scale_kind=SCALE_L2)
    assert sc[0, 0] == np.sqrt(np.float32(1.0 + 2.0 ** -23))
    assert np.float32(np.float32(np.float32(1 + e * e) + e * e) + e * e) == 1.0
    # ... and pairs neighbours, not elements half a block apart: squares (1, 1, h, 2.25h), h = 2^-24,
    # give (1+1) + (h+2.25h) = 2 + 2^-22, while (1+h) + (1+2.25h) = 1 + (1+2h) = 2
    v = np.array([1.0, 1.0, e, 1.5 * e] + [0.0] * 124, dtype=np.float32)
    _, sc = oracle.encode(v[None], None, NORM_NONE, CODEC_QSGD4, B=128, scale_kind=SCALE_L2)
    assert sc[0, 0] == np.sqrt(np.float32(2.0 + 2.0 ** -22))
    # two tiles in one block: the tree runs over the whole block
    v2 = np.concatenate([v, v])
    _, sc = oracle.encode(v2[None], None, NORM_NONE, CODEC_QSGD4, B=256, scale_kind=SCALE_L2)
    assert sc[0, 0] == np.sqrt(np.float32(2 * np.float32(2.0 + 2.0 ** -22)))


def test_zero_elements_never_fire_even_for_tiny_scales():
    # P(z_d = 1) = |v_d| / R = 0 for v_d = 0, whatever u is: with the smallest
    # subnormal as R, u * R rounds to zero for half of all u
    tiny = np.float32(1.4e-45)
    v = np.zeros(512, dtype=np.float32)
    v[::128] = tiny
    for codec in (CODEC_TERN2, CODEC_QSGD4):
        for t in range(3):
            codes, sc = oracle.encode(v[None], None, NORM_NONE, codec, B=128, s=1, t=t)
            out = oracle.decode_aggregate(codes, sc, 512, None, NORM_NONE, codec, B=128, s=1)
            assert np.all(sc == tiny) and not out[v == 0].any()


def test_zero_and_nonfinite_blocks_give_zero_codes():
    g = np.zeros((1, 300), dtype=np.float32)
    g[0, 200] = np.nan
    g[0, 10] = 1.0
    g[0, 150] = 0.0
    codes, sc = oracle.encode(g, None, NORM_NONE, CODEC_SIGN1, B=128)
    out = oracle.decode_aggregate(codes, sc, 300, None, NORM_NONE, CODEC_SIGN1, B=128)
    assert sc[0, 0] == 1.0 and np.isnan(sc[0, 1]) and sc[0, 2] == 0.0
    assert np.all(out[128:] == 0.0) and np.all(codes[0, 4:] == 0)
    g[0, 200] = np.inf
    codes, sc = oracle.encode(g, None, NORM_NONE, CODEC_TERN2, B=128)
    out = oracle.decode_aggregate(codes, sc, 300, None, NORM_NONE, CODEC_TERN2, B=128)
    assert np.isinf(sc[0, 1]) and np.all(out[128:256] == 0.0)


# ------------------------------------------------------------------ normalisation fixed points
@pytest.mark.parametrize("codec", [CODEC_SIGN1, CODEC_TERN2, CODEC_QSGD4])
def test_zero_reference_reduces_to_plain_compression(codec):
    # reference = zeros gives C_nz = 1, the trivial case of Proposition 2
    rng = np.random.default_rng(6)
    g = rng.standard_normal((4, 700)).astype(np.float32)
    zero = np.zeros(700, dtype=np.float32)
    a = oracle.encode(g, zero, NORM_DIFF, codec, B=128, t=5)
    b = oracle.encode(g, None, NORM_NONE, codec, B=128, t=5)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    oa = oracle.decode_aggregate(a[0], a[1], 700, zero, NORM_DIFF, codec, B=128)
    ob = oracle.decode_aggregate(b[0], b[1], 700, None, NORM_NONE, codec, B=128)
    assert np.array_equal(oa, ob)


@pytest.mark.parametrize("codec", [CODEC_SIGN1, CODEC_TERN2, CODEC_QSGD4])
def test_gradient_equal_to_reference_gives_zero_codes(codec):
    # Eq. 2 with g_t = reference: the transmitted difference vanishes and v = reference
    rng = np.random.default_rng(7)
    r = rng.standard_normal(500).astype(np.float32)
    g = np.stack([r, r, r])
    codes, sc = oracle.encode(g, r, NORM_DIFF, codec, B=128)
    assert not codes.any() and not sc.any()
    out = oracle.decode_aggregate(codes, sc, 500, r, NORM_DIFF, codec, B=128)
    assert np.array_equal(out, r)


def test_unit_reference_quotient_equals_plain_compression():
    rng = np.random.default_rng(8)
    g = rng.standard_normal((2, 300)).astype(np.float32)
    ones = np.ones(300, dtype=np.float32)
    a = oracle.encode(g, ones, NORM_QUOT, CODEC_TERN2, B=128, t=2)
    b = oracle.encode(g, None, NORM_NONE, CODEC_TERN2, B=128, t=2)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    oa = oracle.decode_aggregate(a[0], a[1], 300, ones, NORM_QUOT, CODEC_TERN2, B=128)
    ob = oracle.decode_aggregate(b[0], b[1], 300, None, NORM_NONE, CODEC_TERN2, B=128)
    assert np.array_equal(oa, ob)


def test_quotient_of_reference_by_itself_is_full_scale():
    # Eq. 3 with g_t = reference (guard inactive, dyadic values so 1/r and r*(1/r) are exact)
    rng = np.random.default_rng(9)
    r = (2.0 ** rng.integers(-3, 1, size=384) * rng.choice([-1, 1], size=384)).astype(np.float32)
    g = np.stack([r, r])
    codes, sc = oracle.encode(g, r, NORM_QUOT, CODEC_TERN2, B=128)
    assert np.all(sc == 1.0)
    sym = unpack_symbols(codes[0], 384, 2)
    assert np.all(sym == 1)                              # nonzero, positive: v = +R everywhere
    out = oracle.decode_aggregate(codes, sc, 384, r, NORM_QUOT, CODEC_TERN2, B=128)
    assert np.array_equal(out, r)


def test_quotient_guard():
    r = np.zeros(400, dtype=np.float32)
    r[:128] = np.linspace(-1, 1, 128)
    r[5] = 0.0
    r[6] = -0.0
    r[128:256] = 0.0                                     # all-zero tile
    r[256:] = 1e-3
    r[300] = 8.0
    den = oracle.quot_den(r, 2.0 ** -4)
    assert np.all(den[128:256] == 1.0)
    assert np.all(np.abs(den[:128]) >= 2.0 ** -4) and den[5] == 2.0 ** -4 and den[6] == 2.0 ** -4
    big = np.abs(r[:128]) >= 2.0 ** -4
    assert np.array_equal(den[:128][big], r[:128][big])
    assert np.all(np.sign(den[:128][r[:128] < 0]) == -1)
    assert np.all(den[256:384][np.arange(256, 384) != 300] == 0.5) and den[300] == 8.0
    assert np.all(den[384:] == 1e-3 * np.float32(1.0)) or np.all(den[384:] == np.float32(1e-3))


def test_quotient_form_is_unbiased():
    rng = np.random.default_rng(10)
    d, S, M = 256, 1500, 2
    r = (rng.standard_normal(d) * 0.5).astype(np.float32)
    g = (r[None] * (1 + 0.3 * rng.standard_normal((M, d)))).astype(np.float32)
    acc = np.zeros(d)
    for t in range(S):
        codes, sc = oracle.encode(g, r, NORM_QUOT, CODEC_TERN2, B=128, t=t)
        acc += oracle.decode_aggregate(codes, sc, d, r, NORM_QUOT, CODEC_TERN2, B=128)
    mean = acc / S
    gbar = g.astype(np.float64).mean(0)
    den = oracle.quot_den(r).astype(np.float64)
    v = g.astype(np.float64) / den
    Rv = np.stack([np.repeat(np.abs(v[m]).reshape(-1, 128).max(1), 128) for m in range(M)])
    var = (den ** 2 * (Rv * np.abs(v) - v ** 2)).sum(0) / M ** 2
    z = np.abs(mean - gbar) / np.sqrt(var / S + 1e-30)
    assert z.max() < 5.5


# ------------------------------------------------------------------ aggregation
def test_single_worker_difference_decode_adds_reference_back():
    rng = np.random.default_rng(15)
    r = rng.standard_normal(300).astype(np.float32)
    delta = grid_vector(rng, 300, np.float32(0.5), 1)
    g = (r + delta).astype(np.float32)
    codes, sc = oracle.encode(g[None], r, NORM_DIFF, CODEC_TERN2, B=0)
    # v = g - r is not exactly delta in fp32, but it decodes to R * sign * z and out = r + that
    out = oracle.decode_aggregate(codes, sc, 300, r, NORM_DIFF, CODEC_TERN2, B=0)
    plain = oracle.decode_aggregate(codes, sc, 300, None, NORM_NONE, CODEC_TERN2, B=0)
    assert np.array_equal(out, (r + plain).astype(np.float32))


def test_identical_workers_on_grid_points_aggregate_exactly():
    rng = np.random.default_rng(16)
    v = grid_vector(rng, 640, np.float32(2.0), 1)
    for M in [1, 2, 3, 8]:
        g = np.repeat(v[None], M, axis=0)
        codes, sc = oracle.encode(g, None, NORM_NONE, CODEC_TERN2, B=128)
        out = oracle.decode_aggregate(codes, sc, 640, None, NORM_NONE, CODEC_TERN2, B=128)
        if M in (1, 2, 8):
            assert np.array_equal(out, v)
        else:
            assert np.allclose(out, v, rtol=1e-6)


def test_aggregate_is_sequential_fp32_mean_of_single_worker_decodes():
    rng = np.random.default_rng(17)
    M, d = 5, 520
    g = rng.standard_normal((M, d)).astype(np.float32)
    r = (0.9 * g.mean(0)).astype(np.float32)
    codes, sc = oracle.encode(g, r, NORM_DIFF, CODEC_QSGD4, B=256, s=4, t=8)
    out = oracle.decode_aggregate(codes, sc, d, r, NORM_DIFF, CODEC_QSGD4, B=256, s=4)
    singles = [oracle.decode_aggregate(codes[m:m + 1], sc[m:m + 1], d, None, NORM_NONE, CODEC_QSGD4, B=256, s=4)
               for m in range(M)]
    acc = singles[0].copy()
    for m in range(1, M):
        acc = (acc + singles[m]).astype(np.float32)
    want = (r + (acc / np.float32(M)).astype(np.float32)).astype(np.float32)
    assert np.array_equal(out, want)


def test_row_stride_is_honoured():
    rng = np.random.default_rng(18)
    buf = rng.standard_normal((3, 1100)).astype(np.float32)
    view = buf[:, :1000]
    a = oracle.encode(view, None, NORM_NONE, CODEC_TERN2, B=128)
    b = oracle.encode(np.ascontiguousarray(view), None, NORM_NONE, CODEC_TERN2, B=128)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_cnz_of_proposition_2():
    rng = np.random.default_rng(19)
    g = rng.standard_normal((4, 256)).astype(np.float32)
    assert oracle.cnz(g, None) == 1.0                    # reference = zeros: the trivial case
    r = g.mean(0)
    want = ((g.astype(np.float64) - r.astype(np.float64)) ** 2).sum() / (g.astype(np.float64) ** 2).sum()
    assert oracle.cnz(g, r) == pytest.approx(want, rel=1e-12)


@pytest.mark.parametrize("codec", [oracle.CODEC_SIGN1, oracle.CODEC_TERN2, oracle.CODEC_QSGD4])
def test_encoding_a_window_equals_the_window_of_the_whole_encode(codec):
    # coordinates [i0, i0+n) encoded with coord_offset = i0 give exactly the words and scales the
    # whole-vector encode has for those tiles (tiles are independent given the reference)
    d, M, i0, n = 128 * 40 + 17, 3, 128 * 13, 128 * 9
    rng = np.random.default_rng(5)
    g = rng.standard_normal((M, d)).astype(np.float32)
    r = (0.8 * g.mean(0) + 0.1 * rng.standard_normal(d)).astype(np.float32)
    for norm in (oracle.NORM_DIFF, oracle.NORM_QUOT):
        codes, scales = oracle.encode(g, r, norm, codec, B=128, s=5, seed=(7, 1), t=3)
        wc, ws = oracle.encode(np.ascontiguousarray(g[:, i0:i0 + n]), r[i0:i0 + n], norm, codec, B=128, s=5, seed=(7, 1), t=3,
                               coord_offset=i0)
        words = 4 * codec
        assert np.array_equal(wc, codes[:, i0 // 128 * words:(i0 + n) // 128 * words])
        assert np.array_equal(ws.view(np.uint32), scales[:, i0 // 128:(i0 + n) // 128].view(np.uint32))
        # and without the offset the random draws differ
        wc0, _ = oracle.encode(np.ascontiguousarray(g[:, i0:i0 + n]), r[i0:i0 + n], norm, codec, B=128, s=5, seed=(7, 1), t=3)
        assert not np.array_equal(wc0, wc)


# ---- combined form of Section 3: r = Q[(g - ref) ./ ref2], v = ref2 . r + ref -------------------
def _comb_inputs(seed=9, d=128 * 6 + 30, M=4):
    rng = np.random.default_rng(seed)
    g = rng.standard_normal((M, d)).astype(np.float32)
    r = (0.7 * g.mean(0) + 0.2 * rng.standard_normal(d)).astype(np.float32)
    r2 = np.abs(rng.standard_normal(d)).astype(np.float32) + 0.25
    return g, r, r2


def test_combined_form_with_unit_second_reference_is_the_difference_form():
    g, r, _ = _comb_inputs()
    ones = np.ones_like(r)
    for codec in (oracle.CODEC_SIGN1, oracle.CODEC_TERN2, oracle.CODEC_QSGD4):
        a = oracle.encode(g, r, oracle.NORM_COMB, codec, seed=(3, 0), t=2, ref2=ones)
        b = oracle.encode(g, r, oracle.NORM_DIFF, codec, seed=(3, 0), t=2)
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
        oa = oracle.decode_aggregate(a[0], a[1], g.shape[1], r, oracle.NORM_COMB, codec, ref2=ones)
        ob = oracle.decode_aggregate(b[0], b[1], g.shape[1], r, oracle.NORM_DIFF, codec)
        assert np.array_equal(oa, ob)


def test_combined_form_with_zero_first_reference_is_the_quotient_form():
    g, _, r2 = _comb_inputs()
    zeros = np.zeros_like(r2)
    a = oracle.encode(g, zeros, oracle.NORM_COMB, oracle.CODEC_TERN2, seed=(3, 0), t=2, ref2=r2)
    b = oracle.encode(g, r2, oracle.NORM_QUOT, oracle.CODEC_TERN2, seed=(3, 0), t=2)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    oa = oracle.decode_aggregate(a[0], a[1], g.shape[1], zeros, oracle.NORM_COMB, oracle.CODEC_TERN2, ref2=r2)
    ob = oracle.decode_aggregate(b[0], b[1], g.shape[1], r2, oracle.NORM_QUOT, oracle.CODEC_TERN2)
    assert np.array_equal(oa, ob)


def test_combined_form_gradient_equal_to_reference_gives_zero_codes_and_returns_it():
    _, r, r2 = _comb_inputs()
    g = np.repeat(r[None], 3, axis=0)
    codes, scales = oracle.encode(g, r, oracle.NORM_COMB, oracle.CODEC_TERN2, ref2=r2)
    assert not codes.any() and not scales.any()
    out = oracle.decode_aggregate(codes, scales, r.shape[0], r, oracle.NORM_COMB, oracle.CODEC_TERN2, ref2=r2)
    assert np.array_equal(out, r)


def test_combined_form_is_unbiased_and_scales_blocks_by_the_second_reference():
    g, r, r2 = _comb_inputs(d=256, M=1)
    S = 4000
    acc = np.zeros(g.shape[1])
    for t in range(S):
        c, sc = oracle.encode(g, r, oracle.NORM_COMB, oracle.CODEC_TERN2, seed=(1, 2), t=t, ref2=r2)
        acc += oracle.decode_aggregate(c, sc, g.shape[1], r, oracle.NORM_COMB, oracle.CODEC_TERN2, ref2=r2)
    mean = acc / S
    den = oracle.quot_den(r2)
    v = (g[0] - r) / den
    R = np.repeat(np.abs(v).reshape(-1, 128).max(1), 128)
    sigma = den * np.sqrt(np.maximum(R * np.abs(v) - v * v, 0) / S)     # closed-form variance of the ternary code, rescaled
    assert np.all(np.abs(mean - g[0]) <= 5 * sigma + 1e-5)
    # the scale on the wire is max |(g - ref) / den| over the block
    _, sc = oracle.encode(g, r, oracle.NORM_COMB, oracle.CODEC_TERN2, ref2=r2)
    assert np.allclose(sc[0], np.abs(v).reshape(-1, 128).max(1), rtol=1e-6)


def test_magnitude_reference_is_the_mean_absolute_value_of_the_history():
    rng = np.random.default_rng(4)
    hist = [rng.standard_normal(500).astype(np.float32) for _ in range(5)]
    got = oracle.magnitude_reference(hist)
    want = np.mean(np.abs(np.stack(hist).astype(np.float64)), axis=0)
    assert np.allclose(got, want, rtol=1e-6)
    assert np.array_equal(oracle.magnitude_reference([hist[0]]), np.abs(hist[0]))   # k = 1: exactly |h_1|
    st = oracle.State(500, 2, 5, oracle.CODEC_TERN2, oracle.NORM_COMB, fuse_mode=oracle.FUSE_MEAN)
    for h in hist[::-1]:
        st.push_reference(h)
    st.fuse(rng.standard_normal((2, 500)).astype(np.float32))
    assert np.array_equal(st.ref2(), got)
