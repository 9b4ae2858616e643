"""GPU parity, stage level: tng_encode / tng_decode_aggregate through the C ABI
against the CPU oracle on the same seeded inputs and the same reference.
Packed codes, scales and decoded aggregates must match bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import codes_np, make_ctx, round_up4, same_values, to_np
from paper_1901_08227_b200 import tng, workloads

pytestmark = pytest.mark.gpu

CODECS = [tng.CODEC_SIGN1, tng.CODEC_TERN2, tng.CODEC_QSGD4]
NORMS = [tng.NORM_NONE, tng.NORM_DIFF, tng.NORM_QUOT]


def run_both(d, M, codec, norm, B, scale_kind=0, s=7, seed=(3, 9), step=5, ld=None, kind="normal", ref_kind="near"):
    dev = "cuda"
    g = workloads.random_grads(d * 7 + M, M, d, device=dev, ld=ld or round_up4(d), kind=kind)
    if ref_kind == "near":
        ref = (g.mean(0) * 0.9 + 0.05 * workloads.normal((d,), 11, 1, dev)).contiguous()
    elif ref_kind == "zeros":
        ref = torch.zeros(d, device=dev)
    else:   # sparse: whole tiles of zeros and tiny entries, exercises the quotient guard
        ref = g.mean(0).clone()
        ref[: min(d, 200)] = 0.0
        ref[::7] *= 1e-6
        ref = ref.contiguous()
    ctx = make_ctx(d, M, 1, codec, norm, block=B, scale_kind=scale_kind, qsgd_levels=s, seed_lo=seed[0], seed_hi=seed[1])
    ctx.encode(g, ref=ref if norm != tng.NORM_NONE else None, step=step)
    codes, scales = ctx.wire()
    out = torch.empty(d, device=dev)
    ctx.decode_aggregate(out, ref=ref if norm != tng.NORM_NONE else None)
    torch.cuda.synchronize()
    st = ctx.stats()
    gn, rn = to_np(g), to_np(ref)
    oc, osc = oracle.encode(gn, rn if norm != tng.NORM_NONE else None, norm, codec, B=B, s=s, scale_kind=scale_kind,
                            seed=seed, t=step)
    oout = oracle.decode_aggregate(oc, osc, d, rn if norm != tng.NORM_NONE else None, norm, codec, B=B, s=s)
    ctx.close()
    return (codes_np(codes), to_np(scales), to_np(out)), (oc, osc, oout), st


def assert_exact(got, want):
    assert same_values(got[1], want[1]), "scales differ"
    assert np.array_equal(got[0], want[0]), "packed codes differ"
    assert same_values(got[2], want[2]), "decoded aggregate differs"


@pytest.mark.parametrize("codec", CODECS)
@pytest.mark.parametrize("norm", NORMS)
@pytest.mark.parametrize("d,M", [(1, 1), (3, 2), (127, 3), (128, 1), (1000, 4), (4099, 8), (128 * 41, 5)])
def test_block128_bit_exact(codec, norm, d, M):
    got, want, _ = run_both(d, M, codec, norm, 128)
    assert_exact(got, want)


@pytest.mark.parametrize("codec", CODECS)
@pytest.mark.parametrize("scale_kind", [0, 1])
@pytest.mark.parametrize("B,d", [(0, 1000), (0, 5), (256, 65536 // 8 + 77), (384, 3000), (1024, 128 * 50 + 1), (0, 128 * 2100 + 9)])
def test_general_block_sizes_bit_exact(codec, scale_kind, B, d):
    got, want, _ = run_both(d, 3, codec, tng.NORM_DIFF, B, scale_kind=scale_kind, s=4)
    assert_exact(got, want)


@pytest.mark.parametrize("codec", CODECS)
@pytest.mark.parametrize("scale_kind", [0, 1])
@pytest.mark.parametrize("B,d,M,norm", [(256, 2048 * 9 + 50, 8, tng.NORM_DIFF), (512, 2048 * 8, 3, tng.NORM_QUOT),
                                        (1024, 2048 * 11 + 1024 + 384 + 7, 13, tng.NORM_DIFF), (2048, 2048 * 10 + 2047, 5, tng.NORM_NONE),
                                        (256, 2048 * 12 + 128, 64, tng.NORM_QUOT), (2048, 2048 * 150 + 300, 2, tng.NORM_DIFF)])
def test_blocks_of_several_tiles_in_long_vectors_take_one_pass(codec, scale_kind, B, d, M, norm):
    # a scale per 256 .. 2048 coordinates of a vector of at least 8 chunks: the whole chunks go through the
    # staged kernel whose warps share tile statistics, the rest (whole blocks and a ragged one) through
    # the three-launch path; neither wire nor aggregate may show the seam
    got, want, st = run_both(d, M, codec, norm, B, scale_kind=scale_kind, s=6)
    assert st.pipeline_error == 0
    assert_exact(got, want)


@pytest.mark.parametrize("codec", CODECS)
@pytest.mark.parametrize("norm", [tng.NORM_DIFF, tng.NORM_QUOT])
def test_l2_scale_block128(codec, norm):
    got, want, _ = run_both(5000, 4, codec, norm, 128, scale_kind=1)
    assert_exact(got, want)


@pytest.mark.parametrize("codec", CODECS)
@pytest.mark.parametrize("norm,scale_kind,M", [(tng.NORM_NONE, 0, 1), (tng.NORM_DIFF, 0, 8), (tng.NORM_QUOT, 0, 7),
                                               (tng.NORM_DIFF, 1, 16), (tng.NORM_QUOT, 1, 3), (tng.NORM_DIFF, 0, 64)])
@pytest.mark.parametrize("d", [1024 * 17 + 128 * 2 + 77, 2048 * 9 + 128 * 3 + 50])
def test_long_vectors_take_the_staged_kernels(codec, norm, scale_kind, M, d):
    # whole 2048-coordinate chunks go through the bulk-copy pipelines (several fills per
    # chunk when M > 8), the remaining full tiles and the ragged one through the direct
    # kernels: neither the wire nor the aggregate may show the seam.  The second length has
    # a tile count that is a multiple of 4, which the staged decode needs; the first one
    # decodes with the direct kernel.
    got, want, st = run_both(d, M, codec, norm, 128, scale_kind=scale_kind, s=5, ld=d + 7 + (4 - (d + 7) % 4) % 4)
    assert st.pipeline_error == 0
    assert_exact(got, want)


@pytest.mark.parametrize("codec", CODECS)
@pytest.mark.parametrize("scale_kind", [0, 1])
@pytest.mark.parametrize("factor", [1e-28, 1e-33, 1e-38, 3e-42])
def test_tiny_and_subnormal_scales(codec, factor, scale_kind):
    # scales around and below 2^-100 (and subnormal ones): the rounding threshold u*R must be the
    # same correctly rounded product on both sides
    d, M = 2048 * 9 + 128 * 3 + 50, 4
    g = workloads.random_grads(3, M, d, device="cuda", ld=round_up4(d))
    g.mul_(factor)
    g[1, 128 * 5: 128 * 6] *= 1e6                       # one ordinary-looking block among the tiny ones
    ref = (g.mean(0) * 0.5).contiguous()
    ctx = make_ctx(d, M, 1, codec, tng.NORM_DIFF, block=128, seed_lo=1, scale_kind=scale_kind)
    ctx.encode(g, ref=ref, step=3)
    codes, scales = ctx.wire()
    out = torch.empty(d, device="cuda")
    ctx.decode_aggregate(out, ref=ref)
    gn, rn = to_np(g), to_np(ref)
    oc, osc = oracle.encode(gn, rn, tng.NORM_DIFF, codec, B=128, s=7, seed=(1, 0), t=3, scale_kind=scale_kind)
    assert same_values(to_np(scales), osc) and np.array_equal(codes_np(codes), oc)
    assert np.array_equal(to_np(out).view(np.uint32), oracle.decode_aggregate(oc, osc, d, rn, tng.NORM_DIFF, codec, B=128, s=7).view(np.uint32))
    # (with the L2 scale every square underflows below ~1e-23: all scales and all codes are zero then)
    assert oc.any() or (scale_kind == 1 and factor < 1e-28)


@pytest.mark.parametrize("d", [128 * 4, 2048 * 9 + 128 * 3 + 50])
def test_quantiser_level_is_bounded_when_the_l2_scale_falls_short(d):
    # blocks whose only non-zero element has a subnormal square: sqrt(fl(v*v)) < |v|, so s|v|/R > s; the level
    # must stay s and the sign plane must hold the sign (both the direct and the staged kernel)
    M, s = 4, 7
    g = torch.zeros(M, round_up4(d), device="cuda")
    for T in range(0, d // 128, 3):
        g[:, 128 * T + (37 * T) % 128] = torch.tensor([1e-22, 3e-22, -1e-22, -3e-22], device="cuda")
    g[2, 128: 256] = workloads.normal((128,), 5, 2, "cuda")          # an ordinary block among them
    for step in range(6):
        ctx = make_ctx(d, M, 1, tng.CODEC_QSGD4, tng.NORM_NONE, block=128, seed_lo=2, scale_kind=1, qsgd_levels=s)
        ctx.encode(g, step=step)
        codes, scales = ctx.wire()
        out = torch.empty(d, device="cuda")
        ctx.decode_aggregate(out)
        gn = to_np(g)[:, :d]
        oc, osc = oracle.encode(gn, None, tng.NORM_NONE, tng.CODEC_QSGD4, B=128, s=s, seed=(2, 0), t=step, scale_kind=1)
        assert same_values(to_np(scales), osc) and np.array_equal(codes_np(codes), oc)
        want = oracle.decode_aggregate(oc, osc, d, None, tng.NORM_NONE, tng.CODEC_QSGD4, B=128, s=s)
        assert np.array_equal(to_np(out).view(np.uint32), want.view(np.uint32))
        ctx.close()


@pytest.mark.parametrize("s", [1, 2, 3, 4, 5, 6, 7])
def test_qsgd_levels(s):
    got, want, _ = run_both(3001, 4, tng.CODEC_QSGD4, tng.NORM_DIFF, 128, s=s)
    assert_exact(got, want)


@pytest.mark.parametrize("norm", [tng.NORM_DIFF, tng.NORM_QUOT])
@pytest.mark.parametrize("ref_kind", ["zeros", "sparse"])
def test_degenerate_references(norm, ref_kind):
    got, want, _ = run_both(2000, 4, tng.CODEC_TERN2, norm, 128, ref_kind=ref_kind)
    assert_exact(got, want)


def test_heavy_tails_row_stride_and_many_workers():
    got, want, _ = run_both(128 * 64 + 40, 64, tng.CODEC_TERN2, tng.NORM_QUOT, 128, ld=128 * 64 + 44, kind="heavy")
    assert_exact(got, want)
    got, want, _ = run_both(10007, 13, tng.CODEC_SIGN1, tng.NORM_DIFF, 128, ld=10008, kind="heavy")
    assert_exact(got, want)


def test_several_tiles_per_warp_and_seeds():
    # more tiles than resident warps, so every warp loops; several seeds / steps
    d = 128 * 20000 + 17
    for seed, step in [((0, 0), 0), ((0xFFFFFFFF, 7), 123456)]:
        got, want, _ = run_both(d, 2, tng.CODEC_TERN2, tng.NORM_DIFF, 128, seed=seed, step=step)
        assert_exact(got, want)


def test_gradient_equal_to_reference_gives_zero_codes_on_the_gpu():
    d, M = 1500, 3
    r = workloads.normal((d,), 5, 0, "cuda")
    g = r.unsqueeze(0).repeat(M, 1).contiguous()
    ctx = make_ctx(d, M, 1, tng.CODEC_TERN2, tng.NORM_DIFF)
    ctx.encode(g, ref=r, step=0)
    codes, scales = ctx.wire()
    out = torch.empty(d, device="cuda")
    ctx.decode_aggregate(out, ref=r)
    assert not codes.any() and not scales.any()
    assert torch.equal(out, r)


@pytest.mark.parametrize("d", [1000, 2048 * 9 + 128 * 3 + 8])
def test_nonfinite_scales_are_counted_and_zeroed(d):
    M = 2
    g = workloads.random_grads(1, M, d, device="cuda")
    g[0, 300] = float("nan")
    g[1, 700] = float("inf")
    ctx = make_ctx(d, M, 1, tng.CODEC_TERN2, tng.NORM_NONE)
    ctx.encode(g, step=0)
    codes, scales = ctx.wire()
    out = torch.empty(d, device="cuda")
    ctx.decode_aggregate(out)
    gn = to_np(g)
    oc, osc = oracle.encode(gn, None, tng.NORM_NONE, tng.CODEC_TERN2, B=128)
    assert np.array_equal(codes_np(codes), oc) and same_values(to_np(scales), osc)
    assert same_values(to_np(out), oracle.decode_aggregate(oc, osc, d, None, tng.NORM_NONE, tng.CODEC_TERN2, B=128))
    with pytest.raises(tng.TngError) as e:
        ctx.stats(raise_on_nonfinite=True)
    assert e.value.status == tng.ERR_NONFINITE
    assert ctx.stats().nonfinite_scales == 2
    # general block path counts too
    ctx2 = make_ctx(d, M, 1, tng.CODEC_TERN2, tng.NORM_NONE, block=256)
    ctx2.encode(g, step=0)
    assert ctx2.stats().nonfinite_scales == 2


def test_argument_checks_return_status_codes():
    ctx = make_ctx(1000, 2, 1, tng.CODEC_TERN2, tng.NORM_DIFF)
    g = workloads.random_grads(1, 2, 1000, device="cuda")
    buf = torch.zeros(2 * 1002 + 8, device="cuda")
    bad_ld = buf[: 2 * 1002].view(2, 1002)[:, :1000]           # ld = 1002 is not a multiple of 4
    with pytest.raises(tng.TngError) as e:
        ctx.step(bad_ld)
    assert e.value.status == tng.ERR_INVALID_ARG
    misaligned = buf[1: 1 + 2000].view(2, 1000)                # base not 16-byte aligned
    with pytest.raises(tng.TngError) as e:
        ctx.step(misaligned)
    assert e.value.status == tng.ERR_INVALID_ARG
    with pytest.raises(tng.TngError) as e:
        ctx.step_host(torch.zeros(2, 1000), torch.zeros(1000))  # staging was not requested
    assert e.value.status == tng.ERR_STATE
    out = torch.empty(1000, device="cuda")
    ctx.step(g, out)                                            # still usable afterwards
    torch.cuda.synchronize()
    assert torch.isfinite(out).all()
