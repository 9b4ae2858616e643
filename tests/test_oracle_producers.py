"""Pins for the oracle's gradient producers: finite differences of the loss,
closed forms at special points, scipy's Rosenbrock derivative on one pair."""
import numpy as np
import pytest
from scipy.optimize import rosen, rosen_der

import oracle


def test_logistic_gradient_matches_finite_differences():
    rng = np.random.default_rng(0)
    n, d = 40, 9
    X = rng.standard_normal((n, d)).astype(np.float32)
    b = rng.choice([-1.0, 1.0], n).astype(np.float32)
    w = (0.3 * rng.standard_normal(d)).astype(np.float32)
    lam = 0.05
    g = oracle.logistic_grad(X, b, w, lam)
    # central differences on an exactly representable step
    h = 2.0 ** -8
    for j in range(d):
        e = np.zeros(d, dtype=np.float32)
        e[j] = h
        fd = (oracle.logistic_loss(X, b, w + e, lam) - oracle.logistic_loss(X, b, w - e, lam)) / (2 * h)
        assert g[j] == pytest.approx(fd, abs=2e-5)


def test_logistic_closed_forms_at_zero():
    rng = np.random.default_rng(1)
    n, d = 64, 12
    X = rng.standard_normal((n, d)).astype(np.float32)
    b = rng.choice([-1.0, 1.0], n).astype(np.float32)
    w0 = np.zeros(d, dtype=np.float32)
    assert oracle.logistic_loss(X, b, w0, 0.3) == pytest.approx(np.log(2.0), rel=1e-14)
    want = -(b[:, None].astype(np.float64) * X.astype(np.float64)).sum(0) / (2 * n)
    assert np.allclose(oracle.logistic_grad(X, b, w0, 0.3), want, rtol=1e-6, atol=1e-8)
    # the regulariser contributes lambda2 * w
    w = rng.standard_normal(d).astype(np.float32)
    diff = oracle.logistic_grad(X, b, w, 0.5).astype(np.float64) - oracle.logistic_grad(X, b, w, 0.0)
    assert np.allclose(diff, 0.5 * w, atol=1e-6)
    # loss does not overflow for large margins
    assert np.isfinite(oracle.logistic_loss(X * 1e4, b, w, 0.0))


def test_rosenbrock_minimum_and_textbook_derivative():
    ones = np.ones(64, dtype=np.float32)
    assert oracle.rosenbrock_value(ones) == 0.0          # global minimum f(1,1) = 0 of every pair
    assert not oracle.rosenbrock_grad(ones).any()
    rng = np.random.default_rng(2)
    x = rng.uniform(-2, 2, 200).astype(np.float32)
    g = oracle.rosenbrock_grad(x)[0]
    val = 0.0
    for i in range(0, 200, 2):
        pair = x[i:i + 2].astype(np.float64)
        assert np.allclose(g[i:i + 2], rosen_der(pair), rtol=1e-5, atol=1e-3)
        val += rosen(pair)
    assert oracle.rosenbrock_value(x) == pytest.approx(val, rel=1e-12)
    assert np.allclose(g, rosen_der_pairs_fd(x), rtol=1e-3, atol=1e-2)


def rosen_der_pairs_fd(x):
    h = 2.0 ** -10
    out = np.zeros(len(x))
    for j in range(len(x)):
        e = np.zeros(len(x), dtype=np.float32)
        e[j] = h
        out[j] = (oracle.rosenbrock_value(x + e) - oracle.rosenbrock_value(x - e)) / (2 * h)
    return out


def test_rosenbrock_noise_rows_are_added_per_worker():
    rng = np.random.default_rng(3)
    x = rng.uniform(-2, 2, 10).astype(np.float32)
    noise = rng.standard_normal((3, 10)).astype(np.float32)
    g0 = oracle.rosenbrock_grad(x)[0]
    g = oracle.rosenbrock_grad(x, noise)
    assert np.array_equal(g, (g0[None] + noise).astype(np.float32))


def test_sgd_update():
    w = np.array([1.0, -2.0, 0.5], dtype=np.float32)
    v = np.array([4.0, 8.0, -2.0], dtype=np.float32)
    assert np.array_equal(oracle.sgd_update(w, v, 0.25), np.array([0.0, -4.0, 1.0], dtype=np.float32))
