"""The round with the workers spread over ranks (tng_fuse_local / tng_fuse_finish /
tng_encode_local / tng_decode_commit).  Several "ranks" are emulated as several contexts in one
process, the two exchanges done by hand exactly as the collectives would (sum of the statistics
blocks, every rank's wire slots copied to all): all ranks must end up with identical state, equal
to the single-context round -- bit for bit where the reference does not depend on the summation
order of the statistics.  Plus one real NCCL run with a single rank."""
import os

import numpy as np
import pytest
import torch
import torch.distributed as dist

from gpu_util import codes_np, drifting_grads, make_ctx, make_oracle, rel_l2, same_values, to_np
from paper_1901_08227_b200 import distributed, tng

pytestmark = pytest.mark.gpu


def emulated_round(ctxs, grads, t, outs):
    P, M = len(ctxs), grads.shape[0]
    per = M // P
    for p, c in enumerate(ctxs):
        c.fuse_local(grads[p * per:(p + 1) * per])
    total = sum(c.local_stats().clone() for c in ctxs)          # the all-reduce
    for c in ctxs:
        c.local_stats().copy_(total)
        c.fuse_finish()
    for p, c in enumerate(ctxs):
        c.encode_local(grads[p * per:(p + 1) * per], p * per, t)
    blocks = [(c.wire_views()[0][p * per:(p + 1) * per].clone(), c.wire_views()[1][p * per:(p + 1) * per].clone())
              for p, c in enumerate(ctxs)]
    for c in ctxs:                                              # the all-gather
        codes, scales = c.wire_views()
        for p, (bc, bs) in enumerate(blocks):
            codes[p * per:(p + 1) * per].copy_(bc)
            scales[p * per:(p + 1) * per].copy_(bs)
    for c, o in zip(ctxs, outs):
        c.decode_commit(o)


@pytest.mark.parametrize("mode,K", [(tng.FUSE_LAST, 1), (tng.FUSE_MEAN, 3), (tng.FUSE_LSQ, 4), (tng.FUSE_HINDSIGHT, 3)])
@pytest.mark.parametrize("norm,codec,B,d", [(tng.NORM_QUOT, tng.CODEC_TERN2, 128, 2048 * 9 + 128 * 3 + 8),
                                            (tng.NORM_DIFF, tng.CODEC_QSGD4, 256, 3000),
                                            (tng.NORM_COMB, tng.CODEC_SIGN1, 128, 128 * 11 + 4)])
@pytest.mark.parametrize("P", [2, 4])
def test_emulated_ranks_agree_with_each_other_and_with_one_context(mode, K, norm, codec, B, d, P):
    M, steps = 8, 2 * K + 2
    opts = dict(block=B, fuse_mode=mode, seed_lo=6, qsgd_levels=4)
    ranks = [make_ctx(d, M, K, codec, norm, **opts) for _ in range(P)]
    single = make_ctx(d, M, K, codec, norm, **opts)
    orc = make_oracle(d, M, K, codec, norm, **opts)
    outs = [torch.empty(d, device="cuda") for _ in range(P)]
    out1 = torch.empty(d, device="cuda")
    exact = mode in (tng.FUSE_LAST, tng.FUSE_MEAN, tng.FUSE_HINDSIGHT)   # no statistics of the gradients involved
    for t, g in enumerate(drifting_grads(3, steps, M, d, "cuda")):
        emulated_round(ranks, g, t, outs)
        single.step(g, out1)
        want = orc.step(to_np(g))
        for c, o in zip(ranks[1:], outs[1:]):
            assert torch.equal(o, outs[0])
            assert torch.equal(c.wire()[0], ranks[0].wire()[0]) and torch.equal(c.wire()[1], ranks[0].wire()[1])
            assert torch.equal(c.reference(), ranks[0].reference())
        if exact:
            assert torch.equal(outs[0], out1) and torch.equal(ranks[0].wire()[0], single.wire()[0])
            if mode != tng.FUSE_HINDSIGHT:
                assert same_values(to_np(outs[0]), want)
                assert np.array_equal(codes_np(ranks[0].wire()[0]), orc.codes())
        else:
            assert rel_l2(to_np(ranks[0].reference()), to_np(single.reference())) < 1e-5 or t == 0
    st = ranks[0].stats()
    assert st.rounds == steps and st.k == min(steps, K) and st.pipeline_error == 0


def test_least_squares_statistics_are_the_sum_of_the_local_ones():
    d, M, K = 2048 * 9 + 100, 8, 4
    a = make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_DIFF, fuse_mode=tng.FUSE_LSQ)
    b = make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_DIFF, fuse_mode=tng.FUSE_LSQ)
    gs = list(drifting_grads(9, K + 1, M, d, "cuda"))
    for g in gs[:K]:
        a.push_reference(g[0].contiguous())
        b.push_reference(g[0].contiguous())
    g = gs[K]
    a.fuse(g)
    sa = a.stats()
    parts = []
    for lo in (0, 3):                                   # uneven split: 3 + 5 workers
        rows = g[lo:lo + 3] if lo == 0 else g[3:]
        b.fuse_local(rows)
        parts.append(b.local_stats().clone())
    b.local_stats().copy_(parts[0] + parts[1])
    b.fuse_finish()
    sb = b.stats()
    # (the per-coordinate sum over the rows is an fp32 sum on both sides, over 8 rows in one case
    # and over 3 and 5 in the other: agreement to fp32 rounding averaged over d, not to fp64)
    assert np.allclose(np.array(sb.rhs[:K]), np.array(sa.rhs[:K]), rtol=1e-7)
    assert sb.grad_sq == pytest.approx(sa.grad_sq, rel=1e-7)
    assert np.allclose(np.array(sb.alpha[:K]), np.array(sa.alpha[:K]), rtol=0, atol=1e-6)
    assert rel_l2(to_np(b.reference()), to_np(a.reference())) < 1e-6


def test_argument_checks_of_the_local_stages():
    c = make_ctx(1000, 4, 2, tng.CODEC_TERN2, tng.NORM_DIFF)
    g = torch.randn(2, 1000, device="cuda")
    with pytest.raises(tng.TngError) as e:
        c.encode_local(g, 3, 0)                         # workers 3..4 of 4
    assert e.value.status == tng.ERR_INVALID_ARG
    with pytest.raises(tng.TngError) as e:
        c.encode_local(g, 0, 0)                         # no reference yet
    assert e.value.status == tng.ERR_STATE
    c.fuse_local(g)
    c.fuse_finish()
    c.encode_local(g, 2, 0)
    c.decode_commit()
    assert c.stats().rounds == 1


def test_one_rank_over_nccl():
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29533")
    created = not dist.is_initialized()
    if created:
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        d, M, K = 2048 * 9 + 128, 4, 3
        opts = dict(block=128, fuse_mode=tng.FUSE_LSQ, seed_lo=2)
        a = make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_QUOT, **opts)
        b = make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_QUOT, **opts)
        drv = distributed.DistributedRound(a, dist.group.WORLD)
        drv.world = 2                                   # take the collective branches even with one rank
        drv.first, drv.count = 0, M
        out_a, out_b = torch.empty(d, device="cuda"), torch.empty(d, device="cuda")
        for g in drifting_grads(4, 6, M, d, "cuda"):
            drv.step(g, out_a)
            b.step(g, out_b)
            assert rel_l2(to_np(out_a), to_np(out_b)) < 5e-3
        assert a.stats().rounds == 6 and a.stats().pipeline_error == 0
    finally:
        if created:
            dist.destroy_process_group()


# ---------------------------------------------------------------------------------------------
# the other split: every rank holds all workers but a slice of the coordinates
def sliced_round(ctxs, bounds, grads, t, outs):
    for c, (lo, n) in zip(ctxs, bounds):
        c.fuse_local(grads[:, lo:lo + n])
    total = sum(c.local_stats_all().clone() for c in ctxs)      # the all-reduce of Gram, rhs, grad_sq
    for c in ctxs:
        c.local_stats_all().copy_(total)
        c.fuse_finish()
    for c, (lo, n), o in zip(ctxs, bounds, outs):
        c.encode_local(grads[:, lo:lo + n], 0, t)
        c.decode_commit(o)


@pytest.mark.parametrize("mode,K", [(tng.FUSE_LAST, 1), (tng.FUSE_MEAN, 3), (tng.FUSE_LSQ, 4), (tng.FUSE_HINDSIGHT, 3)])
@pytest.mark.parametrize("norm,codec,B,d", [(tng.NORM_QUOT, tng.CODEC_TERN2, 128, 2048 * 40 + 128 * 3 + 8),
                                            (tng.NORM_DIFF, tng.CODEC_QSGD4, 256, 256 * 37 + 100),
                                            (tng.NORM_COMB, tng.CODEC_SIGN1, 128, 128 * 50 + 4)])
@pytest.mark.parametrize("P", [2, 3])
def test_coordinate_slices_reproduce_the_round_over_the_whole_vector(mode, K, norm, codec, B, d, P):
    M, steps = 4, 2 * K + 2
    opts = dict(block=B, fuse_mode=mode, seed_lo=6, qsgd_levels=4)
    bounds = [distributed.coord_range(p, P, d, B) for p in range(P)]
    assert bounds[0][0] == 0 and sum(n for _, n in bounds) == d
    ranks = [make_ctx(n, M, K, codec, norm, coord_offset=lo, **opts) for lo, n in bounds]
    single = make_ctx(d, M, K, codec, norm, **opts)
    orc = make_oracle(d, M, K, codec, norm, **opts)
    outs = [torch.empty(n, device="cuda") for _, n in bounds]
    out1 = torch.empty(d, device="cuda")
    exact = mode in (tng.FUSE_LAST, tng.FUSE_MEAN)               # no statistics involved
    for t, g in enumerate(drifting_grads(3, steps, M, d, "cuda", ld=d + (4 - d % 4) % 4)):
        sliced_round(ranks, bounds, g, t, outs)
        single.step(g, out1)
        want = orc.step(to_np(g))
        whole = torch.cat(outs)
        ref = torch.cat([c.reference() for c in ranks])
        if exact:
            assert torch.equal(whole, out1), f"aggregate differs at round {t}"
            assert same_values(to_np(whole), want)
            codes1, scales1 = single.wire()
            tpb = B // 128
            for c, (lo, n) in zip(ranks, bounds):
                codes, scales = c.wire()
                w0, w1 = lo // 128 * 4 * codec, -(-(lo + n) // 128) * 4 * codec
                assert torch.equal(codes, codes1[:, w0:w1]), f"codes differ at round {t}"
                assert torch.equal(scales, scales1[:, lo // B:-(-(lo + n) // B)])
        else:
            assert rel_l2(to_np(ref), to_np(single.reference())) < 1e-5 or t == 0
            a_s, a_1 = np.array(ranks[0].stats().alpha[:K]), np.array(single.stats().alpha[:K])
            assert np.allclose(a_s, a_1, rtol=0, atol=1e-6 * max(1.0, np.abs(a_1).max()))
            for c in ranks[1:]:                                   # every rank solved the same system
                assert np.array_equal(np.array(c.stats().alpha[:K]), a_s)
    for c in ranks:
        st = c.stats()
        assert st.rounds == steps and st.k == min(steps, K) and st.pipeline_error == 0


def test_a_slice_needs_whole_blocks_and_no_whole_vector_quantities():
    g = torch.randn(2, 1024, device="cuda")
    with pytest.raises(tng.TngError) as e:
        make_ctx(1024, 2, 2, tng.CODEC_TERN2, tng.NORM_DIFF, coord_offset=100)         # not a multiple of 128
    assert e.value.status == tng.ERR_INVALID_ARG
    c = make_ctx(1024, 2, 2, tng.CODEC_TERN2, tng.NORM_DIFF, block=256, coord_offset=128)  # not a multiple of the block
    with pytest.raises(tng.TngError) as e:
        c.step(g)
    assert e.value.status == tng.ERR_INVALID_ARG
    for kw, norm in ((dict(block=0), tng.NORM_DIFF), (dict(block=128), tng.NORM_MEAN)):
        c = make_ctx(1024, 2, 2, tng.CODEC_TERN2, norm, coord_offset=1024, **kw)
        with pytest.raises(tng.TngError) as e:
            c.step(g)
        assert e.value.status == tng.ERR_UNSUPPORTED
    assert distributed.coord_range(1, 2, 1000, 128) == (512, 488)
    with pytest.raises(ValueError):
        distributed.coord_range(3, 4, 300, 128)


@pytest.mark.parametrize("reader", ["reference", "save_state", "decode", "encode_in_two_calls"])
def test_a_reference_still_owed_after_fuse_finish_is_formed_by_whoever_needs_it_first(reader):
    # tng_fuse_finish leaves r = sum alpha_j h_j to the next tng_encode_local.  Whatever else touches the
    # reference first (reading it, saving the state, decoding, an encode of only some of the workers followed by
    # another) must see the same reference and produce the same round as the plain order of calls.
    d, M, K = 2048 * 9 + 128 * 3 + 8, 8, 3
    opts = dict(block=128, fuse_mode=tng.FUSE_MEAN, seed_lo=12)
    a = make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_DIFF, **opts)      # plain order
    b = make_ctx(d, M, K, tng.CODEC_TERN2, tng.NORM_DIFF, **opts)      # with the extra reader
    oa, ob = torch.empty(d, device="cuda"), torch.empty(d, device="cuda")
    for t, g in enumerate(drifting_grads(14, K + 3, M, d, "cuda")):
        a.fuse_local(g)
        a.fuse_finish()
        a.encode_local(g, 0, t)
        a.decode_commit(oa)
        b.fuse_local(g)
        b.fuse_finish()
        if reader == "reference" and t > 0:
            early = b.reference()
        elif reader == "save_state":
            b.save_state()
        elif reader == "decode" and t > 0:
            b.decode_aggregate(ob)                      # decodes the previous wire against the new reference: only must not fault
        if reader == "encode_in_two_calls":
            b.encode_local(g[:3], 0, t)
            b.encode_local(g[3:], 3, t)
        else:
            b.encode_local(g, 0, t)
        b.decode_commit(ob)
        assert torch.equal(oa, ob), f"round {t}"
        assert torch.equal(a.wire()[0], b.wire()[0]) and torch.equal(a.wire()[1], b.wire()[1])
        assert torch.equal(a.reference(), b.reference())
        if reader == "reference" and t > 0:
            assert torch.equal(early, b.reference())
    assert a.stats().rounds == b.stats().rounds == K + 3
