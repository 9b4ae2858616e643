"""GPU parity of the combined normalisation (Section 3, the display after Eq. 3):
r = Q[(g - ref) ./ ref'], v = ref' . r + ref, with ref' the mean absolute value of the stored
aggregates.  Whole rounds against the oracle where the references are exact fp32 on both sides
(delayed-gradient and window-average fusion), stage by stage for the least-squares fusion."""
import numpy as np
import pytest
import torch

from gpu_util import codes_np, drifting_grads, make_ctx, make_oracle, rel_l2, same_values, to_np
from paper_1901_08227_b200 import tng

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode,K", [(tng.FUSE_LAST, 1), (tng.FUSE_LAST, 3), (tng.FUSE_MEAN, 4)])
@pytest.mark.parametrize("codec,B,d,tau", [(tng.CODEC_TERN2, 128, 128 * 9 + 40, 1), (tng.CODEC_SIGN1, 128, 2048 * 9 + 128 * 3 + 8, 1),
                                           (tng.CODEC_QSGD4, 256, 3000, 1), (tng.CODEC_TERN2, 0, 1000, 1),
                                           (tng.CODEC_TERN2, 128, 2048 * 8 + 128 * 7 + 100, 3)])
def test_combined_form_rounds_are_bit_exact(mode, K, codec, B, d, tau):
    M, steps = 4, 7
    opts = dict(block=B, fuse_mode=mode, seed_lo=5, qsgd_levels=4, ref_every=tau)
    ctx = make_ctx(d, M, K, codec, tng.NORM_COMB, **opts)
    orc = make_oracle(d, M, K, codec, tng.NORM_COMB, **opts)
    out = torch.empty(d, device="cuda")
    for t, g in enumerate(drifting_grads(13, steps, M, d, "cuda", ld=d + 4 + (4 - d % 4) % 4)):
        ctx.step(g, out)
        want = orc.step(to_np(g))
        codes, scales = ctx.wire()
        assert same_values(to_np(ctx.reference()), orc.ref()), f"reference differs at round {t}"
        assert np.array_equal(codes_np(codes), orc.codes()), f"codes differ at round {t}"
        assert same_values(to_np(scales), orc.scales())
        assert same_values(to_np(out), want), f"aggregate differs at round {t}"
    assert ctx.stats().pipeline_error == 0


@pytest.mark.parametrize("d", [128 * 30 + 5, 2048 * 10 + 128 * 2 + 60])
def test_combined_form_with_least_squares_fusion_stage_by_stage(d):
    M, K = 4, 4
    opts = dict(block=128, fuse_mode=tng.FUSE_LSQ, seed_lo=8)
    ctx = make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_COMB, **opts)
    orc = make_oracle(d, M, K, tng.CODEC_TERN2, tng.NORM_COMB, **opts)
    out = torch.empty(d, device="cuda")
    for t, g in enumerate(drifting_grads(5, 2 * K + 2, M, d, "cuda")):
        gn = to_np(g)
        ctx.fuse(g)
        orc.fuse(gn)
        oref = orc.ref()
        assert rel_l2(to_np(ctx.reference()), oref) < 1e-5 or not oref.any()
        ref_dev = torch.from_numpy(oref).cuda()
        ctx.encode(g, ref=ref_dev, step=t)                 # the second reference is the context's own: exact
        orc.encode(gn)
        codes, scales = ctx.wire()
        assert np.array_equal(codes_np(codes), orc.codes()), f"codes differ at round {t}"
        assert same_values(to_np(scales), orc.scales())
        ctx.decode_aggregate(out, ref=ref_dev)
        want = orc.decode_push()
        assert same_values(to_np(out), want)
        ctx.push_reference(out)


def test_combined_form_stage_calls_need_a_fusion_first():
    ctx = make_ctx(1000, 2, 2, tng.CODEC_TERN2, tng.NORM_COMB)
    g = torch.randn(2, 1000, device="cuda")
    with pytest.raises(tng.TngError) as e:
        ctx.encode(g, ref=torch.zeros(1000, device="cuda"))
    assert e.value.status == tng.ERR_STATE
    ctx.fuse(g)
    ctx.encode(g)


def test_combined_form_state_resume():
    d, M, K = 2048 * 9 + 128, 3, 3
    opts = dict(block=128, fuse_mode=tng.FUSE_LSQ, seed_lo=3, ref_every=4)
    a = make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_COMB, **opts)
    grads = list(drifting_grads(2, 9, M, d, "cuda"))
    out = torch.empty(d, device="cuda")
    for g in grads[:6]:
        a.step(g, out)
    blob = a.save_state()
    b = make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_COMB, **opts)
    b.load_state(blob)
    out_b = torch.empty(d, device="cuda")
    for g in grads[6:]:
        a.step(g, out)
        b.step(g, out_b)
        assert torch.equal(a.wire()[0], b.wire()[0]) and torch.equal(out, out_b)
