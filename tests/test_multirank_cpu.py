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


def test_algorithmic_bytes_of_the_round():
    per = bench.algorithmic_bytes_per_coord(8, 8, 2, 128, "lsq")
    assert per["dots"] == 64.0 and per["encode"] == 70.25 and per["decode"] == 14.25
    assert sum(per.values()) == 148.5
    split = bench.algorithmic_bytes_per_coord(8, 8, 2, 128, "lsq", ref_in_encode=False)
    assert split["combine"] == 36.0 and split["encode"] == 38.25


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
