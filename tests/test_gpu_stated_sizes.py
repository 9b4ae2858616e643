"""End-to-end parity at the sizes the workloads are stated at (not reduced):

* extended Rosenbrock of Section 4.1 with Gaussian noise per worker: d = 2^20, M = 32 workers, K = 4
  trajectory fusion, difference form, stochastic sign and ternary, 500 steps;
* the dense logistic regression of Section 4.2: d = 65536, M = 16 workers x 2048 samples, column scales
  LogUniform(0.1, 10), 5 % label flips, K = 4 fusion, 4-level quantiser, one scale per 256 coordinates.
  The CPU oracle's producer needs about 5 s per step at this size, so 40 of the 200 steps are run
  (the loss is compared every fifth step and at the end).

Both sides start from the same seeded inputs and never exchange anything afterwards: producer ->
tng_step -> update on the GPU through the C ABI, the same three calls of the oracle on the CPU.
Loss curves must agree to 1e-4 relative."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import make_ctx, make_oracle, to_np
from paper_1901_08227_b200 import tng, workloads

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("codec", [tng.CODEC_SIGN1, tng.CODEC_TERN2])
def test_rosenbrock_at_its_stated_size(codec):
    d, M, K, steps, eta = 1 << 20, 32, 4, 500, 2e-4
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
    st = ctx.stats()
    assert st.rounds == steps and st.pipeline_error == 0 and st.nonfinite_scales == 0
    assert cpu[-1] < cpu[0]
    assert np.max(np.abs(gpu - cpu) / cpu) < 1e-4
    ctx.close()


def test_dense_logistic_regression_at_its_stated_size():
    d, M, n, K, steps, lr, lam = 65536, 16, 2048, 4, 40, 0.05, 1e-4
    free, _ = torch.cuda.mem_get_info()
    if free < 20 * (1 << 30):
        pytest.skip("needs about 20 GiB of free device memory")
    X, b, _ = workloads.logistic_data(0, "cuda", d=d, M=M, n=n, flip=0.05, colscale=(0.1, 10.0))
    Xn, bn = to_np(X), to_np(b)
    opts = dict(block=256, qsgd_levels=4, seed_lo=0)
    ctx = make_ctx(d, M, K, tng.CODEC_QSGD4, tng.NORM_DIFF, **opts)
    orc = make_oracle(d, M, K, tng.CODEC_QSGD4, tng.NORM_DIFF, **opts)
    w = torch.zeros(d, device="cuda")
    wn = np.zeros(d, dtype=np.float32)
    grads = torch.empty((M, d), device="cuda")
    out = torch.empty(d, device="cuda")
    scratch = torch.empty(tng.logistic_scratch_floats(M * n, d), device="cuda")
    loss = torch.zeros(1, dtype=torch.float64, device="cuda")
    Xall, ball = X.reshape(M * n, d), b.reshape(M * n)
    Xn_all, bn_all = Xn.reshape(M * n, d), bn.reshape(M * n)
    gpu, cpu = [], []
    for t in range(steps):
        for m in range(M):
            tng.logistic_grad(X[m], b[m], w, lam, grads[m], scratch)
        ctx.step(grads, out)
        tng.sgd_update(w, out, lr)
        gn = np.stack([oracle.logistic_grad(Xn[m], bn[m], wn, lam) for m in range(M)])
        wn = oracle.sgd_update(wn, orc.step(gn), lr)
        if t % 5 == 4 or t == steps - 1:
            tng.logistic_loss(Xall, ball, w, lam, loss, scratch)
            gpu.append(loss.item())
            cpu.append(oracle.logistic_loss(Xn_all, bn_all, wn, lam))
    gpu, cpu = np.array(gpu), np.array(cpu)
    st = ctx.stats()
    assert st.rounds == steps and st.pipeline_error == 0
    assert cpu[-1] < cpu[0]
    assert np.max(np.abs(gpu - cpu) / cpu) < 1e-4
    ctx.close()
