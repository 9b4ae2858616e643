"""Pins for the oracle's trajectory fusion: Gram statistics, ridge least squares,
the reference combine.  Compared with numpy (float64 matmul, lstsq on the
augmented system) and with closed forms for orthonormal / in-span histories."""
import numpy as np
import pytest

import oracle


def rand_hist(rng, k, d, corr=0.0):
    base = rng.standard_normal(d)
    return [(corr * base + (1 - corr) * rng.standard_normal(d)).astype(np.float32) for _ in range(k)]


@pytest.mark.parametrize("k,M,d", [(1, 1, 7), (3, 4, 1000), (8, 8, 4099), (16, 2, 300)])
def test_fuse_stats_match_float64_matmul(k, M, d):
    rng = np.random.default_rng(k * 100 + M)
    hist = rand_hist(rng, k, d, 0.5)
    buf = rng.standard_normal((M, d + 12)).astype(np.float32)
    grads = buf[:, :d]                                   # strided rows
    G, c, gg = oracle.fuse_stats(hist, grads)
    H = np.stack(hist).astype(np.float64)
    gbar = grads.astype(np.float64).mean(0)
    assert np.allclose(G, H @ H.T, rtol=1e-12)
    assert np.allclose(c, H @ gbar, rtol=1e-10, atol=1e-10)
    assert gg == pytest.approx((grads.astype(np.float64) ** 2).sum() / M, rel=1e-12)
    assert np.array_equal(G, G.T)


@pytest.mark.parametrize("k,d", [(1, 3), (2, 5), (3, 8), (4, 8), (8, 64)])
def test_solve_matches_library_least_squares_on_the_ridge_objective(k, d):
    # alpha minimises sum_m ||g^m - H alpha||^2 + M lambda ||alpha||^2, i.e. the
    # augmented least-squares system [H^T; sqrt(lambda) I] alpha = [gbar; 0]
    rng = np.random.default_rng(k + d)
    hist = rand_hist(rng, k, d, 0.7)
    grads = rng.standard_normal((4, d)).astype(np.float32)
    ridge = 1e-3
    G, c, _ = oracle.fuse_stats(hist, grads)
    a64, a32, flag = oracle.fuse_solve(G, c, ridge)
    assert flag == 0
    H = np.stack(hist).astype(np.float64).T              # d x k
    lam = ridge * np.trace(G) / k
    A = np.vstack([H, np.sqrt(lam) * np.eye(k)])
    rhs = np.concatenate([grads.astype(np.float64).mean(0), np.zeros(k)])
    want = np.linalg.lstsq(A, rhs, rcond=None)[0]
    assert np.allclose(a64, want, rtol=1e-8, atol=1e-10)
    assert np.array_equal(a32, a64.astype(np.float32))
    # stationarity: H^T (gbar - H alpha) = lambda alpha
    assert np.allclose(H.T @ (rhs[:d] - H @ a64), lam * a64, atol=1e-9 * np.abs(G).max())


def test_brute_force_search_cannot_beat_the_solution():
    rng = np.random.default_rng(1)
    hist = rand_hist(rng, 2, 6, 0.3)
    grads = rng.standard_normal((3, 6)).astype(np.float32)
    G, c, _ = oracle.fuse_stats(hist, grads)
    a64, _, _ = oracle.fuse_solve(G, c, 0.0)
    H = np.stack(hist).astype(np.float64)
    g = grads.astype(np.float64)

    def obj(al):
        return sum(((g[m] - al @ H) ** 2).sum() for m in range(3))
    best = obj(a64)
    grid = np.linspace(-0.05, 0.05, 21)
    for da in grid:
        for db in grid:
            assert obj(a64 + np.array([da, db])) >= best - 1e-12


def test_orthonormal_history_and_in_span_gradient():
    rng = np.random.default_rng(2)
    Q, _ = np.linalg.qr(rng.standard_normal((64, 4)))
    hist = [Q[:, j].astype(np.float32) for j in range(4)]
    coeff = np.array([0.5, -2.0, 0.25, 1.5])
    gbar = (np.stack(hist).astype(np.float64).T @ coeff).astype(np.float32)
    grads = np.stack([gbar, gbar])
    G, c, _ = oracle.fuse_stats(hist, grads)
    a64, a32, flag = oracle.fuse_solve(G, c, 0.0)
    assert flag == 0 and np.allclose(a64, coeff, atol=1e-6)
    ref = oracle.combine(hist, a32)
    assert np.allclose(ref, gbar, atol=1e-6)
    # ridge shrinks by 1/(1+lambda) when G = I (lambda = ridge * trace/k = ridge)
    a64r, _, _ = oracle.fuse_solve(np.eye(4), coeff, 0.25)
    assert np.allclose(a64r, coeff / 1.25, rtol=1e-14)


def test_bad_pivot_falls_back_to_the_newest_vector():
    h = np.arange(1, 9, dtype=np.float32)
    G, c, _ = oracle.fuse_stats([h, h.copy(), h.copy()], h[None])
    a64, a32, flag = oracle.fuse_solve(G, c, 0.0)        # rank one, no ridge
    assert flag == 1 and list(a32) == [1.0, 0.0, 0.0]
    a64, a32, flag = oracle.fuse_solve(G, c, 1e-6)       # the ridge makes it solvable
    assert flag == 0 and a64.sum() == pytest.approx(1.0, rel=1e-4)
    z = np.zeros(8, dtype=np.float32)
    G, c, _ = oracle.fuse_stats([z, z], h[None])
    assert oracle.fuse_solve(G, c, 1e-6)[2] == 1


def test_combine_is_an_fp32_fma_chain():
    rng = np.random.default_rng(3)
    hist = rand_hist(rng, 5, 333)
    alpha = rng.standard_normal(5).astype(np.float32)
    ref = oracle.combine(hist, alpha)
    want = alpha.astype(np.float64) @ np.stack(hist).astype(np.float64)
    assert np.allclose(ref, want, rtol=0, atol=4e-7 * np.abs(np.stack(hist)).max() * np.abs(alpha).sum())
    # alpha = e_1 returns the newest vector bit for bit (delayed-gradient reference)
    assert np.array_equal(oracle.combine(hist, np.array([1, 0, 0, 0, 0], dtype=np.float32)), hist[0])
    # exact on dyadic data: window average of past aggregates (Section 3.1, second entry of the pool)
    hd = [(rng.integers(-64, 64, 100) / 32.0).astype(np.float32) for _ in range(4)]
    assert np.array_equal(oracle.combine(hd, np.full(4, 0.25, dtype=np.float32)),
                          (np.stack(hd).astype(np.float64).sum(0) / 4).astype(np.float32))
    # the fused multiply-add keeps the product unrounded: x*x = 1 + 2^-11 + 2^-24 rounds to
    # 1 + 2^-11 in fp32, but fma(x, x, -1) = 2^-11 + 2^-24 exactly
    x = np.float32(1 + 2.0 ** -12)
    got = oracle.combine([np.array([-1.0], dtype=np.float32), np.array([x], dtype=np.float32)],
                         np.array([1.0, x], dtype=np.float32))
    assert got[0] == np.float32(2.0 ** -11 + 2.0 ** -24) and got[0] != np.float32(x * x) - np.float32(1)


def test_hindsight_regression_recovers_a_linear_recurrence():
    # h_t = a h_{t-1} + b h_{t-2}: regressing the newest vector on the older ones and
    # shifting the coefficients by one predicts the next vector exactly
    rng = np.random.default_rng(4)
    a, b = 0.75, -0.5
    seq = [rng.standard_normal(200), rng.standard_normal(200)]
    for _ in range(4):
        seq.append(a * seq[-1] + b * seq[-2])
    hist = [s.astype(np.float32) for s in reversed(seq)][:3]   # newest first
    G, _, _ = oracle.fuse_stats(hist, hist[0][None])
    a64, a32, flag = oracle.fuse_solve_hindsight(G, 0.0)
    assert flag == 0
    pred = oracle.combine(hist, a32)
    nxt = a * seq[-1] + b * seq[-2]
    assert np.allclose(pred, nxt, atol=1e-4)
    assert a64[2] == 0.0 and np.allclose(a64[:2], [a, b], atol=1e-5)
    # fewer than two vectors: delayed-gradient reference
    assert list(oracle.fuse_solve_hindsight(np.array([[2.0]]), 0.0)[1]) == [1.0]
