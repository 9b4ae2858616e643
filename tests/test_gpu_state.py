"""GPU: reference refresh cadence (tng_step with TNG_OPT_REF_EVERY) against the oracle, and
state save / resume (a context that loads a saved state continues bit for bit)."""
import numpy as np
import pytest
import torch

from gpu_util import codes_np, drifting_grads, make_ctx, make_oracle, same_numbers, same_values, to_np
from paper_1901_08227_b200 import tng

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode,K", [(tng.FUSE_LAST, 1), (tng.FUSE_LAST, 3), (tng.FUSE_MEAN, 4)])
@pytest.mark.parametrize("norm,codec,B,d", [(tng.NORM_DIFF, tng.CODEC_TERN2, 128, 128 * 9 + 40),
                                            (tng.NORM_QUOT, tng.CODEC_TERN2, 128, 2048 * 9 + 128 * 3 + 8),
                                            (tng.NORM_DIFF, tng.CODEC_QSGD4, 256, 3000)])
def test_refresh_cadence_matches_the_oracle_bit_for_bit(mode, K, norm, codec, B, d):
    M, steps, tau = 4, 9, 3
    opts = dict(block=B, fuse_mode=mode, seed_lo=2, qsgd_levels=4, ref_every=tau)
    ctx = make_ctx(d, M, K, codec, norm, **opts)
    orc = make_oracle(d, M, K, codec, norm, **opts)
    out = torch.empty(d, device="cuda")
    for t, g in enumerate(drifting_grads(31, steps, M, d, "cuda")):
        ctx.step(g, out)
        want = orc.step(to_np(g))
        codes, scales = ctx.wire()
        # (the delayed-gradient reference is a copy of a ring entry on the GPU and fma(1, h, +0) in the oracle:
        # they differ in the sign of zeros only, which no result depends on)
        same = same_numbers if mode == tng.FUSE_LAST else same_values
        assert same(to_np(ctx.reference()), orc.ref()), f"reference differs at round {t}"
        assert np.array_equal(codes_np(codes), orc.codes()), f"codes differ at round {t}"
        assert same_values(to_np(scales), orc.scales())
        assert same_values(to_np(out), want)
    st = ctx.stats()
    assert st.rounds == steps and st.pipeline_error == 0


@pytest.mark.parametrize("mode,tau", [(tng.FUSE_LSQ, 1), (tng.FUSE_LSQ, 4), (tng.FUSE_LAST, 1), (tng.FUSE_MEAN, 2)])
def test_a_loaded_state_continues_bit_for_bit(mode, tau):
    d, M, K = 2048 * 9 + 128 * 3 + 8, 5, 3
    opts = dict(block=128, fuse_mode=mode, seed_lo=7, seed_hi=1, ref_every=tau)
    a = make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_QUOT, **opts)
    grads = list(drifting_grads(8, 11, M, d, "cuda"))
    out = torch.empty(d, device="cuda")
    for g in grads[:6]:
        a.step(g, out)
    blob = a.save_state()
    assert blob.numel() <= a.state_bytes()
    tail_a = []
    for g in grads[6:]:
        a.step(g, out)
        tail_a.append((a.wire()[0].clone(), a.wire()[1].clone(), out.clone()))
    b = make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_QUOT, **opts)
    b.load_state(blob)
    assert b.stats().rounds == 6 and b.stats().k == K
    for g, (codes, scales, o) in zip(grads[6:], tail_a):
        b.step(g, out)
        assert torch.equal(b.wire()[0], codes) and torch.equal(b.wire()[1], scales) and torch.equal(out, o)
    for j in range(K):
        assert torch.equal(a.history(j), b.history(j))


def test_a_state_of_another_configuration_is_rejected():
    a = make_ctx(1000, 2, 2, tng.CODEC_TERN2, tng.NORM_DIFF, seed_lo=1)
    g = torch.randn(2, 1000, device="cuda")
    a.step(g)
    blob = a.save_state()
    for other in (make_ctx(1000, 2, 2, tng.CODEC_TERN2, tng.NORM_DIFF, seed_lo=2),
                  make_ctx(1000, 2, 2, tng.CODEC_TERN2, tng.NORM_DIFF, seed_lo=1, coord_offset=1024),
                  make_ctx(1000, 2, 3, tng.CODEC_TERN2, tng.NORM_DIFF, seed_lo=1),
                  make_ctx(1004, 2, 2, tng.CODEC_TERN2, tng.NORM_DIFF, seed_lo=1)):
        with pytest.raises(tng.TngError) as e:
            other.load_state(blob)
        assert e.value.status == tng.ERR_INVALID_ARG
    with pytest.raises(tng.TngError) as e:
        a.load_state(blob[:40].clone())
    assert e.value.status == tng.ERR_INVALID_ARG
    small = torch.empty(64, dtype=torch.uint8)
    st = tng.lib().tng_save_state(a._h, small.data_ptr(), small.numel(), None, 0)
    assert st == tng.ERR_ALLOC


def test_a_state_with_the_scalar_reference_continues_bit_for_bit():
    d, M, K = 2048 * 9 + 77, 3, 2
    opts = dict(block=128, seed_lo=3)
    a = make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_MEAN, **opts)
    grads = list(drifting_grads(4, 6, M, d, "cuda"))
    for g in grads:
        g += 0.5                                           # in place: the rows keep their padded stride
    out = torch.empty(d, device="cuda")
    for g in grads[:3]:
        a.step(g, out)
    blob = a.save_state()
    b = make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_MEAN, **opts)
    b.load_state(blob)
    out_b = torch.empty(d, device="cuda")
    for g in grads[3:]:
        a.step(g, out)
        b.step(g, out_b)
        assert torch.equal(out, out_b) and torch.equal(a.wire()[0], b.wire()[0]) and torch.equal(a.wire_means(), b.wire_means())


def test_rounds_on_host_buffers_with_and_without_waiting_agree():
    d, M, K, steps = 2048 * 9 + 333, 3, 2, 5
    opts = dict(block=128, seed_lo=4, host_staging=1)
    a = make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_QUOT, **opts)
    b = make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_QUOT, **opts)
    c = make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_QUOT, block=128, seed_lo=4)
    grads = [g.cpu().contiguous().pin_memory() for g in drifting_grads(6, steps, M, d, "cuda", ld=d)]
    outs_a = [torch.empty(d).pin_memory() for _ in range(steps)]
    outs_b = [torch.empty(d).pin_memory() for _ in range(steps)]
    for g, o in zip(grads, outs_a):
        a.step_host(g, o)
    for g, o in zip(grads, outs_b):
        b.step_host_async(g, o)                            # nothing is waited for until the end
    b.host_wait()
    out = torch.empty(d, device="cuda")
    for g, oa, ob in zip(grads, outs_a, outs_b):
        ld = (d + 3) // 4 * 4
        gd = torch.zeros((M, ld), device="cuda")
        gd[:, :d] = g.cuda()
        c.step(gd[:, :d], out)
        assert torch.equal(oa, ob) and torch.equal(out.cpu(), oa)
    b.host_wait()                                          # nothing pending: returns at once
    assert a.stats().rounds == b.stats().rounds == steps
