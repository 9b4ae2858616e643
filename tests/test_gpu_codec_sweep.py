"""GPU parity on the codec-sweep workload at its smallest size: d = 2^20, M = 8, K = 8, the ring
pre-filled with 8 states of the AR(1) trajectory h_t = 0.9 h_{t-1} + N(0,1), worker gradients
h_t + N(0, sigma^2); 1/2/4-bit codes (4-bit = 7 levels), difference and quotient forms,
one scale per 128 coordinates, least-squares fusion.  Stage by stage: the fused reference
within 1e-5 of the oracle's; wire and aggregate, given the oracle's reference, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import codes_np, make_ctx, make_oracle, rel_l2, same_values, to_np
from paper_1901_08227_b200 import tng, workloads

pytestmark = pytest.mark.gpu

D, M, K = 1 << 20, 8, 8


@pytest.fixture(scope="module")
def trajectory():
    traj = workloads.AR1Trajectory(4, D, device="cuda", rho=0.9)
    hist = [traj.advance().clone() for _ in range(K)]
    traj.advance()
    grads = {sigma: traj.worker_grads(M, sigma) for sigma in (0.1, 1.0)}
    return hist, grads, [to_np(h) for h in hist], {s: to_np(g) for s, g in grads.items()}


@pytest.mark.parametrize("sigma", [0.1, 1.0])
@pytest.mark.parametrize("norm", [tng.NORM_DIFF, tng.NORM_QUOT])
@pytest.mark.parametrize("codec", [tng.CODEC_SIGN1, tng.CODEC_TERN2, tng.CODEC_QSGD4])
def test_codec_sweep_stage_parity(trajectory, codec, norm, sigma):
    hist, grads, hist_np, grads_np = trajectory
    opts = dict(block=128, fuse_mode=tng.FUSE_LSQ, qsgd_levels=7, seed_lo=4, seed_hi=int(sigma * 10))
    ctx = make_ctx(D, M, K, codec, norm, **opts)
    orc = make_oracle(D, M, K, codec, norm, **opts)
    for h, hn in zip(hist, hist_np):
        ctx.push_reference(h)
        orc.push_reference(hn)
    g, gn = grads[sigma], grads_np[sigma]
    ctx.fuse(g)
    orc.fuse(gn)
    st = ctx.stats()
    assert st.solver_fallback == 0 and orc.fallback == 0
    oref = orc.ref()
    assert rel_l2(to_np(ctx.reference()), oref) < 1e-5
    assert np.allclose(np.array(st.alpha[:K]), orc.alpha().astype(np.float64)[:K], rtol=0, atol=1e-5)
    # C_nz of Proposition 2: the innovation of the AR(1) step (1 of variance 1/(1-0.81)) plus the
    # workers' own noise is what the trajectory cannot explain
    assert st.cnz == pytest.approx(oracle.cnz(gn, oref), rel=1e-3)
    assert st.cnz < (0.3 if sigma == 0.1 else 0.5)
    ref_dev = torch.from_numpy(oref).cuda()
    ctx.encode(g, ref=ref_dev, step=0)
    orc.encode(gn)
    codes, scales = ctx.wire()
    assert np.array_equal(codes_np(codes), orc.codes())
    assert same_values(to_np(scales), orc.scales())
    out = torch.empty(D, device="cuda")
    ctx.decode_aggregate(out, ref=ref_dev)
    assert same_values(to_np(out), orc.decode_push())
    assert ctx.stats().pipeline_error == 0
    assert st.bits_per_coord == pytest.approx(codec + 32 / 128 + 64 * K / D)
