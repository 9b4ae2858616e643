"""The N > 1 path of the benchmark on CPU: two `gloo` ranks.  Each rank is an independent TNG
problem (no data-path collective); what the ranks share is the timing rule -- the job is as slow
as its slowest rank -- and the seeding rule -- rank r draws stream r.  The reference arm runs on
rank 0 only."""
import json
import os
import socket
import subprocess
import sys
from pathlib import Path

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))

import bench  # noqa: E402
from paper_1901_08227_b200 import workloads  # noqa: E402


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 3.0 + 2.0 * rank                       # rank 1 is the slow one
    job_ms = bench.max_over_ranks(local_ms, world, "cpu")
    stream = workloads.GradientStream(rank, 4096, 2, device="cpu")
    stream.advance()
    g = stream.worker_grads()
    dist.barrier()
    Path(out_dir, f"rank{rank}.json").write_text(json.dumps({"job_ms": job_ms, "g0": float(g[0, 0]), "gsum": float(g.double().sum())}))
    dist.destroy_process_group()


def test_two_gloo_ranks_share_the_slowest_time_and_draw_their_own_streams(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    r = [json.loads((tmp_path / f"rank{i}.json").read_text()) for i in range(world)]
    assert r[0]["job_ms"] == r[1]["job_ms"] == 5.0
    assert r[0]["gsum"] != r[1]["gsum"]               # different problems per rank
    again = workloads.GradientStream(1, 4096, 2, device="cpu")
    again.advance()
    assert float(again.worker_grads().double().sum()) == r[1]["gsum"]   # reproducible from the rank alone
    # whole-job throughput counts every rank's M x d per step
    assert bench.job_throughput_gbs(2, 8, 1 << 20, 1e-3) == 2 * bench.job_throughput_gbs(1, 8, 1 << 20, 1e-3)


def test_single_rank_needs_no_process_group():
    assert bench.max_over_ranks(1.25, 1, "cpu") == 1.25


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0 and p.stdout.strip() == ""


def test_gpus_flag_starts_its_own_ranks():
    # `bench.py --gpus 2` without a launcher around it starts two ranks itself (what torchrun would do); the
    # --rank-check mode runs that path on CPU: the ranks meet over gloo, agree on the slowest rank's time and
    # assemble a wire block by block, and rank 0 alone prints the line
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    p = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--gpus", "2", "--rank-check"], env=env, capture_output=True,
                       text=True, timeout=300)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [ln for ln in p.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["job_ms"] == 2.0 and line["wire_rows"] == [1, 2]
    # under a launcher (WORLD_SIZE set) the script must not start ranks of its own
    cmd = bench.launch_command(2, ["--gpus", "2"], 29999)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"] and "--nproc-per-node=2" in cmd and cmd[-2:] == ["--gpus", "2"]
    assert "127.0.0.1" in cmd


def test_exchange_bytes_of_the_splits():
    # worker split at the headline shape on 8 ranks: each rank sends its worker's codes and scales, 2^27 * 2 / 8 + 2^20 * 4 bytes
    wpw, nblk = (1 << 27) // 128 * 8, (1 << 27) // 128
    ex = bench.exchange_bytes("workers", 8, 8, wpw, nblk)
    assert ex["allreduce_bytes"] == 136 and ex["allgather_send_bytes_per_rank"] == (1 << 25) + (1 << 22)
    assert ex["allgather_total_bytes"] == 8 * ex["allgather_send_bytes_per_rank"]
    assert bench.exchange_bytes("coords", 4, 8, wpw, nblk) == {"allreduce_bytes": 2184}
    assert bench.exchange_bytes("none", 4, 8, wpw, nblk) == {}


def test_algorithmic_bytes_of_the_round():
    per = bench.algorithmic_bytes_per_coord(8, 8, 2, 128, "lsq")
    assert per["dots"] == 64.0 and per["encode"] == 70.25 and per["decode"] == 14.25
    assert sum(per.values()) == 148.5
    split = bench.algorithmic_bytes_per_coord(8, 8, 2, 128, "lsq", ref_in_encode=False)
    assert split["combine"] == 36.0 and split["encode"] == 38.25
    comb = bench.algorithmic_bytes_per_coord(8, 8, 2, 128, "lsq", norm="comb")     # a second reference written and read
    assert comb["encode"] == 74.25 and comb["decode"] == 18.25
    scalar = bench.algorithmic_bytes_per_coord(8, 8, 2, 128, "lsq", norm="mean")   # no fusion, the rows read twice
    assert set(scalar) == {"encode", "decode"} and scalar["encode"] == 66.25 and scalar["decode"] == 10.25
    last = bench.algorithmic_bytes_per_coord(8, 8, 2, 128, "last")                 # the reference is a ring slot: no combine
    assert "dots" not in last and last["encode"] == 38.25
    # a scale per 256 coordinates is still one read of the rows; one scale per vector needs two
    b256 = bench.algorithmic_bytes_per_coord(16, 4, 4, 256, "lsq", norm="diff")
    assert b256["encode"] == 16 + 64 + 4 + 8 + 0.25
    vec = bench.algorithmic_bytes_per_coord(4, 1, 2, 0, "last", norm="diff")
    assert vec["encode"] == 2 * (16 + 4) + 1.0 and vec["decode"] == 1.0 + 4 + 4 + 4


def _gather_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_1901_08227_b200 import distributed
    M, words = 6, 10
    first, count = distributed.worker_range(rank, world, M)
    wire = torch.zeros((M, words), dtype=torch.int32)
    wire[first:first + count] = torch.arange(first * words, (first + count) * words, dtype=torch.int32).view(count, words)
    dist.all_gather_into_tensor(wire, wire[first:first + count].clone())     # as DistributedRound does, in place
    stats = torch.full((17,), float(rank + 1), dtype=torch.float64)
    dist.all_reduce(stats)
    Path(out_dir, f"wire{rank}.json").write_text(json.dumps({"wire": wire.tolist(), "stats": stats.tolist(), "range": [first, count]}))
    dist.destroy_process_group()


def test_the_wire_exchange_assembles_every_worker_slot_on_every_rank(tmp_path):
    world = 2
    mp.spawn(_gather_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    r = [json.loads((tmp_path / f"wire{i}.json").read_text()) for i in range(world)]
    want = np.arange(60).reshape(6, 10).tolist()
    assert r[0]["wire"] == want and r[1]["wire"] == want          # worker m's words in slot m everywhere
    assert r[0]["stats"] == [3.0] * 17 and r[1]["stats"] == [3.0] * 17
    assert r[0]["range"] == [0, 3] and r[1]["range"] == [3, 3]
    from paper_1901_08227_b200 import distributed
    import pytest
    with pytest.raises(ValueError):
        distributed.worker_range(0, 4, 6)


# ---------------------------------------------------------------------------------------------
# The round with the coordinates split over two gloo ranks.  The rank-local stages are played by
# the oracle on the rank's slice (a stand-in with the context's method names), so that what is
# under test is the driver: which block is all-reduced, in which order the stages run, and that
# the slices put together are the round over the whole vector.
class _OracleSliceContext:
    def __init__(self, first, count, M, K, codec, norm, mode, seed):
        import oracle
        self.o, self.first, self.d, self.M, self.K = oracle, first, count, M, K
        self.codec, self.norm, self.mode, self.seed = codec, norm, mode, seed
        self.hist = []                                     # newest first
        self.block = torch.zeros(273, dtype=torch.float64)
        self.ref = np.zeros(count, dtype=np.float32)
        self.alpha = np.zeros(K, dtype=np.float32)
        self.rounds = 0

    def stats(self):
        from types import SimpleNamespace
        return SimpleNamespace(rounds=self.rounds)

    def fuse_local(self, g):
        self.block.zero_()
        k = len(self.hist)
        if k == 0 or self.mode != self.o.FUSE_LSQ:
            return
        G, c, gg = self.o.fuse_stats(self.hist, g.numpy())   # c and gg are means over the M rows
        blk = self.block.numpy()
        for i in range(k):
            blk[i * 16:i * 16 + k] = G[i]
        blk[256:256 + k] = c * self.M                      # the library hands out raw sums
        blk[272] = gg * self.M

    def local_stats_all(self):
        return self.block

    def fuse_finish(self):
        k = len(self.hist)
        if k == 0:
            self.ref = np.zeros(self.d, dtype=np.float32)
            return
        if self.mode == self.o.FUSE_LSQ:
            blk = self.block.numpy()
            G = np.array([blk[i * 16:i * 16 + k] for i in range(k)])
            _, a32, _ = self.o.fuse_solve(G, blk[256:256 + k] / self.M, 1e-6)
        else:                                              # window average
            a32 = np.full(k, np.float32(1.0) / np.float32(k), dtype=np.float32)
        self.alpha = a32
        self.ref = self.o.combine(self.hist, a32)

    def encode_local(self, g, m_first, step):
        assert m_first == 0
        self.wire = self.o.encode(g.numpy(), self.ref, self.norm, self.codec, B=128, seed=(self.seed, 0), t=step,
                                  coord_offset=self.first)

    def decode_commit(self, out):
        codes, scales = self.wire
        res = self.o.decode_aggregate(codes, scales, self.d, self.ref, self.norm, self.codec, B=128)
        self.hist = ([res] + self.hist)[:self.K]
        self.rounds += 1
        if out is not None:
            out.copy_(torch.from_numpy(res))


def _sliced_main(rank, world, port, out_dir, mode):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_1901_08227_b200 import distributed
    d, M, K, steps = 128 * 21 + 50, 3, 3, 6
    first, count = distributed.coord_range(rank, world, d, 128)
    ctx = _OracleSliceContext(first, count, M, K, oracle.CODEC_TERN2, oracle.NORM_DIFF, mode, seed=4)
    drv = distributed.CoordShardedRound(ctx, group=dist.group.WORLD)
    rng = np.random.default_rng(0)                         # the same gradients on both ranks
    outs, alphas = [], []
    mean = rng.standard_normal(d).astype(np.float32)
    for t in range(steps):
        if t == 3:   # a driver created in mid-run takes the round number (the Philox step) from the context
            drv = distributed.CoordShardedRound(ctx, group=dist.group.WORLD)
            assert drv.round == 3
        mean = (0.9 * mean + 0.3 * rng.standard_normal(d)).astype(np.float32)
        g = (mean[None] + 0.5 * rng.standard_normal((M, d))).astype(np.float32)
        out = torch.empty(count)
        drv.step(torch.from_numpy(np.ascontiguousarray(g[:, first:first + count])), out)
        outs.append(out.numpy().copy())
        alphas.append(ctx.alpha.copy())
    np.save(Path(out_dir, f"sliced{rank}.npy"), np.stack(outs))
    np.save(Path(out_dir, f"alpha{rank}.npy"), np.stack([np.resize(a, K) for a in alphas]))
    dist.destroy_process_group()


def _whole_vector_rounds(mode):
    import oracle
    d, M, K, steps = 128 * 21 + 50, 3, 3, 6
    st = oracle.State(d, M, K, oracle.CODEC_TERN2, oracle.NORM_DIFF, fuse_mode=mode, seed_lo=4)
    rng = np.random.default_rng(0)
    outs = []
    mean = rng.standard_normal(d).astype(np.float32)
    for t in range(steps):
        mean = (0.9 * mean + 0.3 * rng.standard_normal(d)).astype(np.float32)
        g = (mean[None] + 0.5 * rng.standard_normal((M, d))).astype(np.float32)
        outs.append(st.step(g))
    return np.stack(outs)


def test_coordinate_slices_over_two_gloo_ranks_make_the_whole_round(tmp_path):
    import oracle
    world = 2
    for mode in (oracle.FUSE_MEAN, oracle.FUSE_LSQ):
        mp.spawn(_sliced_main, args=(world, _free_port(), str(tmp_path), mode), nprocs=world, join=True)
        got = np.concatenate([np.load(tmp_path / f"sliced{r}.npy") for r in range(world)], axis=1)
        want = _whole_vector_rounds(mode)
        a0, a1 = np.load(tmp_path / "alpha0.npy"), np.load(tmp_path / "alpha1.npy")
        assert np.array_equal(a0, a1)                      # both ranks solved the summed statistics
        if mode == oracle.FUSE_MEAN:
            assert np.array_equal(got, want)               # no statistics: bit for bit
        else:
            # the Gram is summed slice by slice, so alpha may differ in the last bits: close, not equal
            rel = np.linalg.norm(got.astype(np.float64) - want) / np.linalg.norm(want)
            assert rel < 0.05 and np.array_equal(got[0], want[0])       # round 0: empty ring, exact
            assert np.abs(a0).max() > 0.1                  # the statistics did arrive (alpha is not zero)


def test_coordinate_ranges_are_whole_blocks_that_cover_the_vector():
    from paper_1901_08227_b200 import distributed
    import pytest
    for d, world, block in ((1000, 2, 128), (128 * 9, 3, 256), (1 << 20, 8, 128), (129, 2, 128)):
        spans = [distributed.coord_range(r, world, d, block) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][0] + spans[-1][1] == d
        for (lo, n), (lo2, _) in zip(spans, spans[1:]):
            assert lo + n == lo2 and lo2 % block == 0
    with pytest.raises(ValueError):
        distributed.coord_range(0, 2, 1000, 100)
    with pytest.raises(ValueError):
        distributed.coord_range(1, 2, 128, 128)
