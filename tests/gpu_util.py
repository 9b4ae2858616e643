"""Helpers of the GPU parity tests: move seeded inputs to both sides."""
import numpy as np
import torch

import oracle
from paper_1901_08227_b200 import tng, workloads


def round_up4(d):
    return (d + 3) // 4 * 4


def to_np(t):
    return t.detach().cpu().numpy()


def codes_np(t):
    return to_np(t).view(np.uint32)


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return np.linalg.norm(a - b) / (den if den > 0 else 1.0)


def same_bits(a, b):
    """float arrays equal bit for bit (NaN payloads included), +0 == -0 not tolerated"""
    return np.array_equal(np.asarray(a, dtype=np.float32).view(np.uint32), np.asarray(b, dtype=np.float32).view(np.uint32))


def same_values(a, b):
    """float arrays equal bit for bit (+0 and -0 differ), except that a NaN equals a NaN whatever its payload"""
    a = np.ascontiguousarray(a, dtype=np.float32)
    b = np.ascontiguousarray(b, dtype=np.float32)
    if a.shape != b.shape:
        return False
    return bool(np.all((a.view(np.uint32) == b.view(np.uint32)) | (np.isnan(a) & np.isnan(b))))


def same_numbers(a, b):
    """equal as numbers (+0 == -0), NaN == NaN"""
    return np.array_equal(np.asarray(a), np.asarray(b), equal_nan=True)


def make_ctx(d, M, K, codec, norm, **opts):
    return tng.Context(d, M, K, codec, norm, **opts)


def make_oracle(d, M, K, codec, norm, **opts):
    opts = {k: v for k, v in opts.items() if k not in ("timing", "host_staging")}
    return oracle.State(d, M, K, codec, norm, **opts)


def drifting_grads(seed, steps, M, d, device, ld=None, noise=0.3):
    """slowly drifting mean + per-worker noise, as (M, d) views with row stride ld"""
    traj = workloads.AR1Trajectory(seed, d, device=device, rho=0.95)
    if ld is None:
        ld = round_up4(d)
    for _ in range(steps):
        traj.advance()
        yield traj.worker_grads(M, noise, ld=ld)
