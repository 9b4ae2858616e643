"""GPU parity of the gradient producers and of short end-to-end optimisation runs
(producer -> tng_step -> parameter update) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import make_ctx, make_oracle, rel_l2, same_values, to_np
from paper_1901_08227_b200 import tng, workloads

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n,d", [(500, 1000), (37, 129), (256, 4096), (64, 10)])
def test_logistic_gradient_and_loss(n, d):
    X, b, _ = workloads.logistic_data(3, "cuda", d=d, M=1, n=n, colscale=(0.1, 10.0))
    X, b = X[0].contiguous(), b[0].contiguous()
    w = 0.1 * workloads.normal((d,), 4, 0, "cuda")
    scratch = torch.empty(tng.logistic_scratch_floats(n, d), device="cuda")
    grad = torch.empty(d, device="cuda")
    loss = torch.zeros(1, dtype=torch.float64, device="cuda")
    tng.logistic_grad(X, b, w, 1e-3, grad, scratch)
    tng.logistic_loss(X, b, w, 1e-3, loss, scratch)
    want_g = oracle.logistic_grad(to_np(X), to_np(b), to_np(w), 1e-3)
    want_l = oracle.logistic_loss(to_np(X), to_np(b), to_np(w), 1e-3)
    assert rel_l2(to_np(grad), want_g) < 1e-5
    assert loss.item() == pytest.approx(want_l, rel=1e-6)


def test_rosenbrock_gradient_is_bit_exact_and_value_matches():
    d, M = 2 * 5001, 5
    x = workloads.rosenbrock_x0(1, d, "cuda")
    noise = workloads.rosenbrock_noise(1, 0, M, d, "cuda")
    grads = torch.empty((M, d), device="cuda")
    val = torch.zeros(1, dtype=torch.float64, device="cuda")
    tng.rosenbrock_grad(x, noise, grads)
    tng.rosenbrock_value(x, val)
    assert same_values(to_np(grads), oracle.rosenbrock_grad(to_np(x), to_np(noise)))
    assert val.item() == pytest.approx(oracle.rosenbrock_value(to_np(x)), rel=1e-12)
    tng.rosenbrock_grad(x, None, grads)
    assert same_values(to_np(grads), np.repeat(oracle.rosenbrock_grad(to_np(x)), M, axis=0))
    w = x.clone()
    tng.sgd_update(w, grads[0].contiguous(), 2e-4)
    assert same_values(to_np(w), oracle.sgd_update(to_np(x), to_np(grads[0]), 2e-4))


def run_logistic(d, M, n, K, codec, B, s, steps, lr, lam, colscale, flip, fuse_mode=tng.FUSE_AUTO, seed=0):
    X, b, _ = workloads.logistic_data(seed, "cuda", d=d, M=M, n=n, flip=flip, colscale=colscale)
    Xn, bn = to_np(X), to_np(b)
    opts = dict(block=B, qsgd_levels=s, seed_lo=seed, fuse_mode=fuse_mode)
    ctx = make_ctx(d, M, K, codec, tng.NORM_DIFF, **opts)
    orc = make_oracle(d, M, K, codec, tng.NORM_DIFF, **opts)
    w = torch.zeros(d, device="cuda")
    wn = np.zeros(d, dtype=np.float32)
    grads = torch.empty((M, d), device="cuda")
    out = torch.empty(d, device="cuda")
    scratch = torch.empty(tng.logistic_scratch_floats(n, d), device="cuda")
    loss = torch.zeros(1, dtype=torch.float64, device="cuda")
    Xall, ball = X.reshape(M * n, d), b.reshape(M * n)
    gpu_curve, cpu_curve = [], []
    for t in range(steps):
        for m in range(M):
            tng.logistic_grad(X[m], b[m], w, lam, grads[m], scratch)
        ctx.step(grads, out)
        tng.sgd_update(w, out, lr)
        scratch_all = torch.empty(tng.logistic_scratch_floats(M * n, d), device="cuda")
        tng.logistic_loss(Xall, ball, w, lam, loss, scratch_all)
        gpu_curve.append(loss.item())
        gn = np.stack([oracle.logistic_grad(Xn[m], bn[m], wn, lam) for m in range(M)])
        wn = oracle.sgd_update(wn, orc.step(gn), lr)
        cpu_curve.append(oracle.logistic_loss(Xn.reshape(M * n, d), bn.reshape(M * n), wn, lam))
    return np.array(gpu_curve), np.array(cpu_curve)


def test_tiny_logistic_regression_loss_curve():
    # d=1000, M=4 x 500 samples, 10% flips, difference form, reference = last aggregate (K=1),
    # ternary with one scale per vector, 50 gradient steps, lr 0.1
    gpu, cpu = run_logistic(1000, 4, 500, 1, tng.CODEC_TERN2, 0, 7, 50, 0.1, 1e-4, None, 0.10)
    assert cpu[-1] < cpu[0]
    assert np.max(np.abs(gpu - cpu) / cpu) < 1e-4


def test_dense_logistic_regression_loss_curve_reduced():
    # the dense configuration (K=4 fusion, 4-level quantiser, block 256) at a size the oracle
    # finishes in seconds: d=4096, M=4 x 256 samples, column scales LogUniform(0.1, 10), 5% flips
    gpu, cpu = run_logistic(4096, 4, 256, 4, tng.CODEC_QSGD4, 256, 4, 40, 0.05, 1e-4, (0.1, 10.0), 0.05)
    assert cpu[-1] < cpu[0]
    assert np.max(np.abs(gpu - cpu) / cpu) < 1e-4


@pytest.mark.parametrize("codec", [tng.CODEC_SIGN1, tng.CODEC_TERN2])
def test_rosenbrock_loss_curve_reduced(codec):
    # extended Rosenbrock, noise N(0, 0.1^2) per worker, K=4 fusion, block 128, eta 2e-4
    d, M, K, steps, eta = 1 << 14, 8, 4, 60, 2e-4
    ctx = make_ctx(d, M, K, codec, tng.NORM_DIFF, seed_lo=3)
    orc = make_oracle(d, M, K, codec, tng.NORM_DIFF, seed_lo=3)
    x = workloads.rosenbrock_x0(2, d, "cuda")
    xn = to_np(x).copy()
    grads = torch.empty((M, d), device="cuda")
    out = torch.empty(d, device="cuda")
    val = torch.zeros(1, dtype=torch.float64, device="cuda")
    gpu, cpu = [], []
    for t in range(steps):
        noise = workloads.rosenbrock_noise(2, t, M, d, "cuda")
        tng.rosenbrock_grad(x, noise, grads)
        ctx.step(grads, out)
        tng.sgd_update(x, out, eta)
        tng.rosenbrock_value(x, val)
        gpu.append(val.item())
        gn = oracle.rosenbrock_grad(xn, to_np(noise))
        xn = oracle.sgd_update(xn, orc.step(gn), eta)
        cpu.append(oracle.rosenbrock_value(xn))
    gpu, cpu = np.array(gpu), np.array(cpu)
    assert cpu[-1] < cpu[0]
    assert np.max(np.abs(gpu - cpu) / cpu) < 1e-4
