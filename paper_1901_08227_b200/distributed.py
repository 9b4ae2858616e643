"""Workers spread over GPUs: one process per GPU (``torch.distributed``, NCCL), every process a
``tng.Context`` of the same configuration and the gradient rows of its own workers.

A round is the rank-local stages of the library with two exchanges between them (Algorithm 1:
every server codes its gradient, the codes are exchanged, everyone decodes the same average):

    fuse_local -> all-reduce of 17 doubles -> fuse_finish -> encode_local
               -> all-gather of the wire (codes and scales) -> decode_commit

(with the scalar reference of Section 3.1 the fusion stages drop out and the workers' scalars
are gathered with the wire).

Only plumbing lives here; every computation is a library call.  The collectives run on the
wire and statistics buffers in place (zero-copy views of the context's workspace), which are
this GPU's own memory.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import tng


def worker_range(rank: int, world: int, M: int):
    """Workers [first, first + count) of `rank`: M must split evenly over the ranks so that the
    wire can be all-gathered as equal blocks."""
    if M % world != 0:
        raise ValueError(f"M = {M} workers do not split evenly over {world} ranks")
    count = M // world
    return rank * count, count


class _StageClock:
    """Optional CUDA-event marks between the stages of a round (on the current stream, which is the one
    the library calls are given): mean milliseconds per stage over the rounds since start_timing()."""

    def __init__(self, names):
        self.names, self.marks = names, None

    def start(self):
        self.marks = []

    def mark(self):
        if self.marks is not None:
            ev = torch.cuda.Event(enable_timing=True)
            ev.record()
            self.marks.append(ev)

    def times(self):
        n = len(self.names) + 1
        if not self.marks or len(self.marks) < n:
            return {}
        torch.cuda.synchronize()
        rounds = len(self.marks) // n
        out = {name: 0.0 for name in self.names}
        for r in range(rounds):
            evs = self.marks[r * n:(r + 1) * n]
            for i, name in enumerate(self.names):
                out[name] += evs[i].elapsed_time(evs[i + 1]) / rounds
        return out


class DistributedRound:
    """Drives one context per rank.  `group` may be None (a single process: no exchange)."""

    STAGES = ("statistics", "exchange_statistics", "solve_combine", "encode", "exchange_wire", "decode")

    def __init__(self, ctx: tng.Context, group=None):
        self.ctx, self.group = ctx, group
        self.world = dist.get_world_size(group) if group is not None else 1
        self.rank = dist.get_rank(group) if group is not None else 0
        self.first, self.count = worker_range(self.rank, self.world, ctx.M)
        self.clock = _StageClock(self.STAGES)
        self.resync()

    def resync(self):
        """Take the round number (the Philox step) from the context: it is ahead of zero after a
        loaded state or earlier rounds, and the codes must use the context's own counter."""
        self.round = int(self.ctx.stats().rounds)

    def step(self, local_grads: torch.Tensor, out: torch.Tensor | None = None):
        """local_grads: (count, d) rows of this rank's workers.  Returns `out` (the aggregate)."""
        if local_grads.shape[0] != self.count:
            raise ValueError(f"rank {self.rank} owns {self.count} workers, got {local_grads.shape[0]} rows")
        ctx, clock = self.ctx, self.clock
        scalar_ref = ctx.norm == tng.NORM_MEAN          # every worker's own scalar: no fusion, no statistics
        clock.mark()
        if not scalar_ref:
            ctx.fuse_local(local_grads)
        clock.mark()
        if not scalar_ref and self.world > 1:
            dist.all_reduce(ctx.local_stats(), op=dist.ReduceOp.SUM, group=self.group)
        clock.mark()
        if not scalar_ref:
            ctx.fuse_finish()
        clock.mark()
        ctx.encode_local(local_grads, self.first, self.round)
        clock.mark()
        if self.world > 1:
            codes, scales = ctx.wire_views()
            lo, hi = self.first, self.first + self.count
            dist.all_gather_into_tensor(codes, codes[lo:hi].clone(), group=self.group)
            dist.all_gather_into_tensor(scales, scales[lo:hi].clone(), group=self.group)
            if scalar_ref:                               # the scalars travel with the codes
                means = ctx.wire_means_view()
                dist.all_gather_into_tensor(means, means[lo:hi].clone(), group=self.group)
        clock.mark()
        ctx.decode_commit(out)
        clock.mark()
        self.round += 1
        return out


def coord_range(rank: int, world: int, d: int, block: int = 128):
    """Coordinates [first, first + count) of `rank` when every rank holds a slice of all vectors:
    slices are whole scale blocks (multiples of 128 coordinates), the last one takes the ragged end."""
    if block < 128 or block % 128 != 0:
        raise ValueError("slices need a scale block that is a multiple of 128 coordinates")
    units = -(-d // block)
    per = -(-units // world)
    first = min(rank * per * block, d)
    count = min(first + per * block, d) - first
    if count <= 0:
        raise ValueError(f"d = {d} is too short for {world} ranks of whole {block}-coordinate blocks")
    return first, count


class CoordShardedRound:
    """The other split: every rank holds all M workers but only its slice of the coordinates (ring
    and wire included).  `ctx` is a context of the slice's length created with
    ``coord_offset=first`` (so that it draws the random numbers of its coordinates of the whole
    vector).  Coding and decoding are local; the fusion statistics are sums over coordinates:

        fuse_local -> all-reduce of 273 doubles (Gram, rhs, grad_sq) -> fuse_finish
                   -> encode_local (all M workers) -> decode_commit

    Every rank ends up with its slice of what one context over the whole vector computes."""

    STAGES = ("statistics", "exchange_statistics", "solve_combine", "encode", "decode")

    def __init__(self, ctx: tng.Context, group=None):
        self.ctx, self.group = ctx, group
        self.world = dist.get_world_size(group) if group is not None else 1
        self.clock = _StageClock(self.STAGES)
        self.resync()

    def resync(self):
        """Take the round number (the Philox step) from the context, see DistributedRound.resync."""
        self.round = int(self.ctx.stats().rounds)

    def step(self, grads_slice: torch.Tensor, out: torch.Tensor | None = None):
        """grads_slice: (M, count) — this rank's coordinates of every worker's gradient."""
        ctx = self.ctx
        if grads_slice.shape[0] != ctx.M:
            raise ValueError(f"expected the rows of all {ctx.M} workers, got {grads_slice.shape[0]}")
        clock = self.clock
        clock.mark()
        ctx.fuse_local(grads_slice)
        clock.mark()
        if self.world > 1:
            dist.all_reduce(ctx.local_stats_all(), op=dist.ReduceOp.SUM, group=self.group)
        clock.mark()
        ctx.fuse_finish()
        clock.mark()
        ctx.encode_local(grads_slice, 0, self.round)
        clock.mark()
        ctx.decode_commit(out)
        clock.mark()
        self.round += 1
        return out
