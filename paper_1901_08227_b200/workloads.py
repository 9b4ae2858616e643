"""Seeded synthetic inputs shaped like the paper's workloads (Section 4).

This module only draws random inputs.  It holds none of the method's arithmetic
(no normalisation, coding, fusion or gradient formulas) and is imported neither
by the CUDA binding nor by the CPU oracle: tests and the benchmark call it and
hand the same buffers to both sides.

Every generator takes a ``device``; values are drawn on that device with a
``torch.Generator`` seeded from ``seed`` and a per-call stream id, and are copied
to the host by the caller when the oracle needs them.
"""
from __future__ import annotations

import math

import torch


def _gen(seed: int, stream: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((int(seed) * 1000003 + int(stream)) % (2 ** 63 - 1))
    return g


def normal(shape, seed, stream=0, device="cpu", std=1.0, mean=0.0):
    out = torch.empty(shape, dtype=torch.float32, device=device)
    out.normal_(mean, std, generator=_gen(seed, stream, device))
    return out


def uniform(shape, lo, hi, seed, stream=0, device="cpu"):
    out = torch.empty(shape, dtype=torch.float32, device=device)
    out.uniform_(lo, hi, generator=_gen(seed, stream, device))
    return out


def log_uniform(shape, lo, hi, seed, stream=0, device="cpu"):
    return torch.exp(uniform(shape, math.log(lo), math.log(hi), seed, stream, device))


def padded_rows(rows: torch.Tensor, ld: int) -> torch.Tensor:
    """Copy an (M, d) tensor into the first d columns of an (M, ld) buffer and
    return the (M, d) strided view (row stride ld)."""
    M, d = rows.shape
    buf = torch.zeros((M, ld), dtype=rows.dtype, device=rows.device)
    buf[:, :d] = rows
    return buf[:, :d]


# --------------------------------------------------------------------------- logistic regression
def logistic_data(seed, device="cpu", d=1000, M=4, n=500, flip=0.10, colscale=None):
    """Features N(0,1) (optionally times a per-column scale drawn LogUniform
    (colscale=(lo,hi))), labels sign(x.w*) with w*~N(0,I) and a fraction ``flip``
    of them negated.  Returns X[M,n,d], b[M,n] in {-1,+1}, scale[d] or None."""
    X = normal((M, n, d), seed, 1, device)
    scale = None
    if colscale is not None:
        scale = log_uniform((d,), colscale[0], colscale[1], seed, 2, device)
        X = X * scale
    wstar = normal((d,), seed, 3, device)
    b = torch.sign(X @ wstar)
    b = torch.where(b == 0, torch.ones_like(b), b)
    flips = uniform((M, n), 0.0, 1.0, seed, 4, device) < flip
    b = torch.where(flips, -b, b)
    return X.contiguous(), b.contiguous(), scale


# --------------------------------------------------------------------------- extended Rosenbrock
def rosenbrock_x0(seed, d, device="cpu"):
    return uniform((d,), -2.0, 2.0, seed, 10, device)


def rosenbrock_noise(seed, step, M, d, device="cpu", sigma=0.1):
    """Per-worker additive gradient noise N(0, sigma^2) of one step."""
    return normal((M, d), seed, 1000 + step, device, std=sigma)


# --------------------------------------------------------------------------- AR(1) trajectory (codec sweep)
class AR1Trajectory:
    """h_t = rho h_{t-1} + N(0,1); worker grads = h_t + N(0, sigma^2)."""

    def __init__(self, seed, d, device="cpu", rho=0.9):
        self.seed, self.d, self.device, self.rho = seed, d, device, rho
        self.t = 0
        self.h = normal((d,), seed, 20, device)

    def advance(self):
        self.t += 1
        self.h = self.rho * self.h + normal((self.d,), self.seed, 20 + self.t, self.device)
        return self.h

    def worker_grads(self, M, sigma, ld=None):
        rows = self.h.unsqueeze(0) + normal((M, self.d), self.seed, 5000 + self.t, self.device, std=sigma)
        return rows.contiguous() if ld is None else padded_rows(rows, ld)


# --------------------------------------------------------------------------- DNN-sized gradient stream
class GradientStream:
    """Heavy-tailed gradients around a slowly drifting mean.

    The d coordinates form ``segments`` equal "layers"; layer scale ~
    LogUniform(1e-4, 1e-1).  mu_0 = scale.N(0,1); mu_t = rho mu_{t-1} +
    sqrt(1-rho^2) scale.N(0,1).  Worker gradient = mu_t + scale.T with T
    Student-t (nu=3), drawn as z / sqrt(chi2_3 / 3)."""

    def __init__(self, seed, d, M, device="cpu", segments=64, rho=0.99, nu=3):
        self.seed, self.d, self.M, self.device, self.rho, self.nu = seed, d, M, device, rho, nu
        seg = log_uniform((segments,), 1e-4, 1e-1, seed, 30, device)
        reps = (d + segments - 1) // segments
        self.scale = seg.repeat_interleave(reps)[:d].contiguous()
        self.t = 0
        self.mu = self.scale * normal((d,), seed, 31, device)

    def advance(self):
        self.t += 1
        eps = normal((self.d,), self.seed, 31 + self.t, self.device)
        self.mu = self.rho * self.mu + math.sqrt(1.0 - self.rho ** 2) * self.scale * eps
        return self.mu

    def worker_grads(self, out=None, first=0, count=None):
        """Rows of workers first .. first + count - 1 (default: all M).  A worker's row depends on
        (seed, step, worker) only, so ranks that hold different workers draw consistent rows."""
        count = self.M - first if count is None else count
        if out is None:
            out = torch.empty((count, self.d), dtype=torch.float32, device=self.device)
        for r in range(count):
            m = first + r
            stream = 100000 + self.t * 128 + m
            z = normal((self.d,), self.seed, stream, self.device)
            chi = torch.zeros_like(z)
            for q in range(self.nu):
                w = normal((self.d,), self.seed, stream + 50000000 * (q + 1), self.device)
                chi.addcmul_(w, w)
            chi.div_(float(self.nu)).sqrt_()
            z.div_(chi).mul_(self.scale).add_(self.mu)
            out[r].copy_(z)
        return out


def random_grads(seed, M, d, device="cpu", ld=None, kind="normal"):
    """Generic (M, d) gradient rows for unit tests; row stride ld if given."""
    if kind == "normal":
        rows = normal((M, d), seed, 40, device)
    elif kind == "heavy":
        z = normal((M, d), seed, 41, device)
        w = normal((M, d), seed, 42, device)
        rows = z / (w.abs() + 0.05)
    else:
        raise ValueError(kind)
    return rows.contiguous() if ld is None else padded_rows(rows, ld)
