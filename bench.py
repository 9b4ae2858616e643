#!/usr/bin/env python
"""Benchmark of the TNG round (tng_step) on synthetic data shaped like a DNN-sized
gradient stream: d = 2^27 fp32 coordinates, M = 8 workers, ring depth K = 8,
quotient normalisation, ternary codes with one scale per 128 coordinates.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  `value` is GB/s of fp32 gradient (all M workers) pushed
through whole rounds with inputs resident in device memory; `e2e` is the same
metric through tng_step_host_async / tng_host_wait (pinned host buffers, both
copies of every round inside the timed region; the blocking tng_step_host is
reported beside it); `roofline` describes the dominant kernel; `cpu_baseline` is the CPU
oracle timed on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

METRIC = "TNG step GB/s of fp32 gradient (all M workers)"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

WORKLOADS = {
    # the headline: a DNN-sized gradient stream
    "c5_dnn_stream": dict(d=1 << 27, M=8, K=8, norm="quot", codec="tern2", block=128, fuse="lsq", levels=7, inputs="stream"),
    "c5_mid": dict(d=1 << 24, M=8, K=8, norm="quot", codec="tern2", block=128, fuse="lsq", levels=7, inputs="stream"),   # profiler-sized
    "c5_small": dict(d=1 << 22, M=8, K=8, norm="quot", codec="tern2", block=128, fuse="lsq", levels=7, inputs="stream"),
    # the optimisation workloads: tng_step only, gradients from the producers outside the timed region
    "c1_tiny": dict(d=1000, M=4, K=1, norm="diff", codec="tern2", block=0, fuse="last", levels=7, inputs="logistic",
                    n=500, flip=0.10, colscale=None, lr=0.1),
    "c2_dense": dict(d=65536, M=16, K=4, norm="diff", codec="qsgd4", block=256, fuse="lsq", levels=4, inputs="logistic",
                     n=2048, flip=0.05, colscale=(0.1, 10.0), lr=0.05),
    "c3_rosenbrock": dict(d=1 << 20, M=32, K=4, norm="diff", codec="tern2", block=128, fuse="lsq", levels=7, inputs="rosenbrock",
                          lr=2e-4),
    # one point of the codec sweep (AR(1) trajectory); --workload c4_sweep runs them all
    "c4_point": dict(d=1 << 24, M=8, K=8, norm="diff", codec="tern2", block=128, fuse="lsq", levels=7, inputs="ar1", sigma=0.1),
}
L2_BYTES = 126e6
FLUSH_BYTES = 256 << 20            # written between timed rounds when a round's inputs would stay in L2
SINGLE_PASS_BLOCKS = (128, 256, 512, 1024, 2048)   # scale blocks the encode pass handles in one read of the rows


def algorithmic_bytes_per_coord(M, K, bits, block, fuse, user_out=True, ref_in_encode=True, norm="quot"):
    """Bytes per coordinate each kernel of one round has to move (reads + writes).

    dots    reads the K ring rows and the M gradient rows;
    encode  reads the M gradient rows and writes the wire (codes + scales); with the reference
            combine folded into it it also reads the K ring rows and writes the reference,
            otherwise it reads the reference a separate combine pass wrote; a scale block that the
            pass cannot finish in one read (one scale per vector, blocks that are not 128 * 2^j <= 2048)
            costs a second read of the rows and of the reference;
    decode  reads the wire and the reference, writes the new ring entry (and the caller's copy).
    The combined form carries a second reference wherever the first one is read or written; the
    scalar reference has no fusion at all, its encode reads the gradient rows twice (means, then codes)."""
    beff = block if block else float("inf")
    wire = M * bits / 8.0 + 4.0 * M / beff
    passes = 1.0 if block in SINGLE_PASS_BLOCKS else 2.0
    per = {}
    if norm == "mean":
        per["encode"] = 4.0 * M * (1.0 + passes) + wire
        per["decode"] = wire + 4.0 + (4.0 if user_out else 0.0)
        return per
    refs = 8.0 if norm == "comb" else (0.0 if norm == "none" else 4.0)
    if fuse == "lsq":
        per["dots"] = 4.0 * K + 4.0 * M
    elif fuse == "hindsight":
        per["dots"] = 4.0 * K                      # Gram of the ring only
    combines = fuse != "last" and norm != "none"   # the delayed-gradient reference is a ring slot as it is
    if combines and ref_in_encode:
        per["encode"] = 4.0 * K + refs + passes * 4.0 * M + (passes - 1.0) * refs + wire
    else:
        if combines:
            per["combine"] = 4.0 * K + refs
        per["encode"] = passes * (4.0 * M + refs) + wire
    per["decode"] = wire + refs + 4.0 + (4.0 if user_out else 0.0)
    return per


# dram__bytes_read.sum + dram__bytes_write.sum per coordinate of the dominant kernel, from the ncu
# capture summarised under profiles/ (taken at d = 2^24 and scaled by d: every kernel streams each
# coordinate once).  None = the kernel changed after the capture.
# integer/logic-pipe instructions the staged encode kernel issues per tile and worker (ternary, quotient
# form; from the opcode histogram of the same capture: 22 logic ops, 9 float compares, 8 ballots, 6 integer
# compares, 4 conversions, 3 integer adds, 3 max, 2 selects, 3 others)
ALU_PIPE_INSTR_PER_TILE_WORKER = 60
NCU_TRAFFIC_BYTES_PER_COORD = {"encode": 69.89, "dots": 64.24, "decode": 11.19}


def measured_hbm_peak():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index, period=0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for name, bit in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def enum_of(tng, cfg):
    norm = {"none": tng.NORM_NONE, "diff": tng.NORM_DIFF, "quot": tng.NORM_QUOT, "comb": tng.NORM_COMB,
            "mean": tng.NORM_MEAN}[cfg["norm"]]
    codec = {"sign1": tng.CODEC_SIGN1, "tern2": tng.CODEC_TERN2, "qsgd4": tng.CODEC_QSGD4}[cfg["codec"]]
    fuse = {"lsq": tng.FUSE_LSQ, "last": tng.FUSE_LAST, "mean": tng.FUSE_MEAN, "hindsight": tng.FUSE_HINDSIGHT}[cfg["fuse"]]
    return norm, codec, fuse


INPUT_RECIPES = {
    "stream": "Student-t(nu=3) around an AR(1) mean (rho 0.99), 64 segments with LogUniform(1e-4,1e-1) scales",
    "ar1": "reference trajectory h_t = 0.9 h_{t-1} + N(0,1), worker gradients h_t + N(0, sigma^2)",
    "logistic": "logistic-regression gradients (N(0,1) features, optional LogUniform column scales, flipped labels) of a short "
                "optimisation run; the producers run outside the timed region",
    "rosenbrock": "extended-Rosenbrock gradients + N(0, 0.1^2) per worker of a short optimisation run; the producer runs "
                  "outside the timed region",
}
SHARDING = {
    "none": "one process per GPU, each rank an independent problem of the full size (no data-path collective)",
    "workers": "the M workers spread over the ranks (Algorithm 1's servers): all-reduce of 17 doubles, then all-gather of "
               "the wire into each GPU's own memory; every rank decodes the same aggregate",
    "coords": "every rank holds all M workers and a slice of whole scale blocks of every vector: one all-reduce of 273 doubles",
}


def config_dict(name, cfg, world, split="none", flushed=False):
    c = {"workload": name, "d": cfg["d"], "M": cfg["M"], "K": cfg["K"], "normalisation": cfg["norm"],
         "codec": cfg["codec"], "block": cfg["block"], "fusion": cfg["fuse"],
         "stream": INPUT_RECIPES[cfg.get("inputs", "stream")],
         "l2": ("L2 flushed between timed rounds (a %d MiB buffer is rewritten; each round timed by its own events)" % (FLUSH_BYTES >> 20))
               if flushed else "inputs exceed L2: every round streams the whole ring and all M gradient rows from HBM",
         "sharding": SHARDING[split] if (world > 1 or split != "none") else "single GPU"}
    if cfg["codec"] == "qsgd4":
        c["levels"] = cfg.get("levels", 7)
    if "sigma" in cfg:
        c["sigma"] = cfg["sigma"]
    return c


def max_over_ranks(value, world, device):
    """The slowest rank's time: every rank gets max_r value_r (the job is as slow as that rank)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    if world > 1 or (dist.is_available() and dist.is_initialized()):
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.item()


def job_throughput_gbs(world, M, d, seconds_per_step):
    """GB/s of fp32 gradient of the whole job: every rank pushes its own M x d problem per step."""
    return world * M * d * 4 / seconds_per_step / 1e9


def exchange_bytes(split, world, M, wpw, nblk):
    """Bytes one rank sends per round in the two splits (what crosses the links; received = (world - 1) x sent for
    the all-gather, the all-reduce is 136 / 2184 bytes whatever the algorithm)."""
    if split == "workers":
        share = (M // world) * (wpw + nblk) * 4
        return {"allreduce_bytes": 17 * 8, "allgather_send_bytes_per_rank": share, "allgather_total_bytes": share * world}
    if split == "coords":
        return {"allreduce_bytes": 273 * 8}
    return {}


# --------------------------------------------------------------------------------------
def run_reference(args, name, cfg):
    """The CPU oracle, as it stands, timed on a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np

    import oracle
    from paper_1901_08227_b200 import tng, workloads
    norm, codec, fuse = enum_of(tng, cfg)
    M, K = cfg["M"], cfg["K"]
    d_s = min(cfg["d"], 1 << 22)                  # the sample: the first 2^22 coordinates of the stream
    stream = workloads.GradientStream(0, d_s, M, device="cpu")
    orc = oracle.State(d_s, M, K, codec, norm, block=cfg["block"], fuse_mode=fuse, qsgd_levels=cfg.get("levels", 7))
    for _ in range(K):
        orc.push_reference(stream.advance().numpy())
    batches = []
    for _ in range(2):
        stream.advance()
        batches.append(stream.worker_grads().numpy())
    for w in range(args.warmup):
        orc.step(batches[w % 2])
    t0 = time.perf_counter()
    for s in range(args.steps):
        orc.step(batches[s % 2])
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    value = M * d_s * 4 / dt / 1e9
    cores = oracle.omp_threads()
    sample = f"first {d_s} of {cfg['d']} coordinates per step (same stream recipe, M={M}, K={K})"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": config_dict(name, cfg, 1),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def time_cpu_baseline(cfg, enums, limit_s=12.0, single_thread=True):
    import numpy as np

    import oracle
    from paper_1901_08227_b200 import workloads
    norm, codec, fuse = enums
    M, K = cfg["M"], cfg["K"]
    d_s = min(cfg["d"], 1 << 22)
    stream = workloads.GradientStream(0, d_s, M, device="cpu")
    orc = oracle.State(d_s, M, K, codec, norm, block=cfg["block"], fuse_mode=fuse, qsgd_levels=cfg.get("levels", 7))
    for _ in range(K):
        orc.push_reference(stream.advance().numpy())
    stream.advance()
    g = stream.worker_grads().numpy()
    orc.step(g)                                    # warm-up (page faults, thread pool)
    n, t0 = 0, time.perf_counter()
    while True:
        orc.step(g)
        n += 1
        dt = time.perf_counter() - t0
        if dt > limit_s or n >= 50:
            break
    per = dt / n
    cores = oracle.omp_threads()
    res = {"value": M * d_s * 4 / per / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": f"first {d_s} of {cfg['d']} coordinates per step (gradient-stream recipe, same M, K, codec, block), {n} steps, {per * 1e3:.1f} ms each"}
    if single_thread and cores > 1:
        # the same oracle on one thread, on a shorter sample (a quarter of the coordinates, one step)
        d_1 = min(d_s, max(d_s // 4, 1 << 14))
        orc1 = oracle.State(d_1, M, K, codec, norm, block=cfg["block"], fuse_mode=fuse, qsgd_levels=cfg.get("levels", 7))
        for j in range(K):
            orc1.push_reference(np.ascontiguousarray(orc.history(K - 1 - j)[:d_1]))
        g1 = np.ascontiguousarray(g[:, :d_1])
        oracle.set_threads(1)
        try:
            t1 = time.perf_counter()
            orc1.step(g1)
            dt1 = time.perf_counter() - t1
        finally:
            oracle.set_threads(cores)
        res["single_thread"] = {"value": M * d_1 * 4 / dt1 / 1e9, "unit": UNIT,
                                "sample": f"first {d_1} coordinates, 1 step, {dt1 * 1e3:.0f} ms"}
    return res


# --------------------------------------------------------------------------------------
def make_problem(tng, workloads, cfg, enums, dev, rank, world, split, extra_opts):
    """Context with its ring filled and two gradient batches, all resident on the device.
    Returns (ctx, driver or None, batches, out)."""
    import torch
    norm, codec, fuse = enums
    d, M, K = cfg["d"], cfg["M"], cfg["K"]
    opts = dict(block=cfg["block"], fuse_mode=fuse, qsgd_levels=cfg.get("levels", 7))
    opts.update(extra_opts)
    kind = cfg.get("inputs", "stream")
    seed = rank if split == "none" else 0           # split problems: every rank sees the same trajectory
    first, count, c_first, c_count = 0, M, 0, d
    if split == "workers":
        from paper_1901_08227_b200 import distributed
        first, count = distributed.worker_range(rank, world, M)
    elif split == "coords":
        from paper_1901_08227_b200 import distributed
        c_first, c_count = distributed.coord_range(rank, world, d, max(cfg["block"], 128))
        opts["coord_offset"] = c_first
    ctx = tng.Context(c_count, M, K, codec, norm, seed_lo=seed, **opts)
    batches = []
    if kind in ("stream", "ar1"):
        if kind == "stream":
            src = workloads.GradientStream(seed, d, M, device=dev)
            rows = lambda: src.worker_grads(first=first, count=count)
        else:
            src = workloads.AR1Trajectory(seed, d, device=dev)
            rows = lambda: src.worker_grads(M, cfg.get("sigma", 0.1))[first:first + count]
        for _ in range(K):
            ctx.push_reference(src.advance()[c_first:c_first + c_count].contiguous())
        for _ in range(2):
            src.advance()
            g = rows()
            batches.append(g[:, c_first:c_first + c_count].contiguous() if split == "coords" else g)
        del src
    else:
        if split != "none":
            raise SystemExit("the optimisation workloads are single-context problems: use --split none")
        # a short optimisation run fills the ring with real aggregates; its last two gradient batches are the timed inputs
        grads = torch.empty((M, d), device=dev)
        agg = torch.empty(d, device=dev)
        if kind == "logistic":
            X, b, _ = workloads.logistic_data(seed, dev, d=d, M=M, n=cfg["n"], flip=cfg["flip"], colscale=cfg["colscale"])
            w = torch.zeros(d, device=dev)
            scratch = torch.empty(tng.logistic_scratch_floats(cfg["n"], d), device=dev)
            def produce(t):
                for m in range(M):
                    tng.logistic_grad(X[m], b[m], w, 1e-4, grads[m], scratch)
        else:
            w = workloads.rosenbrock_x0(seed, d, dev)
            def produce(t):
                tng.rosenbrock_grad(w, workloads.rosenbrock_noise(seed, t, M, d, dev), grads)
        for t in range(K + 2):
            produce(t)
            if t >= K:
                batches.append(grads.clone())
            ctx.step(grads, agg)
            tng.sgd_update(w, agg, cfg["lr"])
        torch.cuda.synchronize()
        if kind == "logistic":
            del X, b, scratch
    driver = None
    if split == "workers":
        driver = distributed.DistributedRound(ctx, group=torch.distributed.group.WORLD if world > 1 else None)
    elif split == "coords":
        driver = distributed.CoordShardedRound(ctx, group=torch.distributed.group.WORLD if world > 1 else None)
    out = torch.empty(c_count, device=dev)
    torch.cuda.empty_cache()
    return ctx, driver, batches, out


def timed_rounds(torch, step, steps, barrier, local, flush_buf):
    """Time `steps` calls of step(i) with CUDA events on the current stream, the clocks sampled meanwhile.
    With flush_buf every round is bracketed by its own events and the buffer is rewritten in between
    (untimed); otherwise one pair of events brackets all rounds.  Returns (ms per round, clocks)."""
    sampler = ClockSampler(local)
    sampler.start()
    barrier()
    if flush_buf is None:
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for i in range(steps):
            step(i)
        ev1.record()
        barrier()
        total = ev0.elapsed_time(ev1)
    else:
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for i in range(steps):
            flush_buf.add_(1)
            evs[i][0].record()
            step(i)
            evs[i][1].record()
        barrier()
        total = sum(a.elapsed_time(b) for a, b in evs)
    return total / steps, sampler.stop()


def stage_split(st0, st1, per_coord, d, peak, sm_mhz):
    """Per-kernel mean duration over the rounds between two tng_stats snapshots (events the library
    records on the launching stream), with GB/s of algorithmic bytes and kilocycles at the sampled clock."""
    n0, n1 = st0.timed_rounds, st1.timed_rounds
    def stage_ms(field):
        return (getattr(st1, field) * n1 - getattr(st0, field) * n0) / max(n1 - n0, 1)
    kernels = {}
    for kname, field in (("dots", "ms_dots"), ("combine", "ms_combine"), ("encode", "ms_encode"), ("decode", "ms_decode")):
        if kname not in per_coord:
            continue
        ms = stage_ms(field)
        gbs = per_coord[kname] * d / (ms * 1e-3) / 1e9 if ms > 0 else None
        kernels[kname] = {"ms": ms, "bytes_per_coord": per_coord[kname], "GBps": gbs, "frac_of_measured": gbs / peak if gbs else None}
        if sm_mhz:
            kernels[kname]["kcycles"] = ms * sm_mhz            # ms x MHz = thousands of SM cycles
    kernels["solve"] = {"ms": stage_ms("ms_solve")}
    return kernels, stage_ms("ms_combine")


def run_ours(args, name, cfg, emit=True):
    import torch
    import torch.distributed as dist

    from paper_1901_08227_b200 import tng, workloads

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    launched = world > 1 or "TORCHELASTIC_RUN_ID" in os.environ     # under torchrun, also with one rank
    if launched and not dist.is_initialized():
        dist.init_process_group("nccl", device_id=dev)
    tng.lib()                                       # fail loudly if libtng.so is missing

    enums = enum_of(tng, cfg)
    norm, codec, fuse = enums
    d, M, K = cfg["d"], cfg["M"], cfg["K"]
    bits = codec
    split = args.split

    cpu_baseline = None
    if rank == 0 and not args.no_cpu_baseline:
        cpu_baseline = time_cpu_baseline(cfg, enums)

    ctx, driver, batches, out = make_problem(tng, workloads, cfg, enums, dev, rank, world, split, dict(timing=1))
    d_local = ctx.d
    if driver is None:
        step = lambda i: ctx.step(batches[i % 2], out)
    else:
        step = lambda i: driver.step(batches[i % 2], out)

    def barrier():
        if launched:
            dist.barrier()
        torch.cuda.synchronize()

    # a round whose inputs (ring + gradient rows) are not well beyond L2 needs the cache flushed between rounds
    round_inputs = (K + batches[0].shape[0]) * d_local * 4
    flush_buf = torch.zeros(FLUSH_BYTES // 4, device=dev) if round_inputs < 2 * L2_BYTES else None

    for w in range(args.warmup):
        step(w)
    barrier()
    st0 = ctx.stats()
    if driver is not None:
        driver.clock.start()        # the split rounds are timed stage by stage by the driver (events between its calls)
    ms_local, clocks = timed_rounds(torch, step, args.steps, barrier, local, flush_buf)
    ms_step = max_over_ranks(ms_local, world, dev)
    st1 = ctx.stats()
    launches = st1.kernel_launches - st0.kernel_launches

    peak, peak_src = measured_hbm_peak()
    _, combine_ms = stage_split(st0, st1, {}, d_local, peak, None)
    # (in the rank-local rounds the first tng_encode_local after a fusion forms the reference, as tng_step's encode does)
    ref_in_encode = cfg["norm"] not in ("none", "mean") and cfg["fuse"] != "last" and (driver is not None or combine_ms == 0.0)
    per_coord = algorithmic_bytes_per_coord(M if split != "workers" else M // world, K, bits, cfg["block"], cfg["fuse"],
                                            ref_in_encode=ref_in_encode, norm=cfg["norm"])
    if split == "workers":     # every rank still decodes all M workers' codes
        full = algorithmic_bytes_per_coord(M, K, bits, cfg["block"], cfg["fuse"], ref_in_encode=ref_in_encode, norm=cfg["norm"])
        per_coord["decode"] = full["decode"]
    kernels, _ = stage_split(st0, st1, per_coord, d_local, peak, clocks.get("sm_mhz"))
    if driver is not None:
        # rank-local stages: statistics = dots, solve_combine = tng_fuse_finish (the solve; the combine is left to the encode)
        stage_ms = driver.clock.times()
        driver.clock.marks = None
        kernels = {}
        for sname, key in (("statistics", "dots"), ("encode", "encode"), ("decode", "decode")):
            if key in per_coord and stage_ms.get(sname):
                ms = stage_ms[sname]
                gbs = per_coord[key] * d_local / (ms * 1e-3) / 1e9
                kernels[key] = {"ms": ms, "bytes_per_coord": per_coord[key], "GBps": gbs, "frac_of_measured": gbs / peak}
        kernels["solve"] = {"ms": stage_ms.get("solve_combine", 0.0)}
        kernels["exchanges"] = {k: v for k, v in stage_ms.items() if k.startswith("exchange")}
    if ref_in_encode and "encode" in kernels:
        kernels["encode"]["includes"] = "reference combine (ring rows -> reference) folded into the encode pass"
    dominant = max((k for k in kernels if "bytes_per_coord" in kernels[k]), key=lambda k: kernels[k]["ms"])
    # the counters were taken on the headline configuration; any other one has no capture
    profiled = split == "none" and all(cfg[k] == WORKLOADS["c5_dnn_stream"][k] for k in ("M", "K", "norm", "codec", "block", "fuse"))
    tpc = NCU_TRAFFIC_BYTES_PER_COORD.get(dominant) if profiled else None
    traffic = tpc * d if tpc is not None else None
    roofline = {"bound": "hbm", "kernel": dominant, "achieved": kernels[dominant]["GBps"], "peak": peak, "unit": "GB/s",
                "frac": kernels[dominant]["frac_of_measured"], "peak_source": peak_src, "traffic": traffic,
                "algorithmic_bytes_per_launch": per_coord[dominant] * d_local}
    if profiled and dominant == "encode" and clocks.get("sm_mhz"):
        # The encode pass is the one kernel that is closer to an arithmetic roof than to HBM: its busiest unit
        # is the integer/logic pipe, which takes one warp instruction every two cycles per SM partition
        # (4 partitions x 148 SMs).  The opcode histogram of the ncu capture gives the number of such
        # instructions per tile (128 coordinates) and worker; stated beside the HBM figure, not instead of it.
        alu_peak = 0.5 * 4 * 148 * clocks["sm_mhz"] * 1e6
        alu_rate = ALU_PIPE_INSTR_PER_TILE_WORKER * (d / 128.0) * M / (kernels["encode"]["ms"] * 1e-3)
        roofline["alu_pipe"] = {"bound": "alu", "achieved": alu_rate / 1e9, "peak": alu_peak / 1e9, "unit": "G warp-instr/s",
                                "frac": alu_rate / alu_peak,
                                "peak_source": "0.5 warp-instr/cycle x 4 partitions x 148 SMs x sampled SM clock"}
    step_bytes = sum(v for k, v in per_coord.items()) * d_local
    step_gbs = step_bytes / (ms_step * 1e-3) / 1e9

    # ---- the same rounds for long enough that the power-limited clock is reached (a short burst runs at the top clock)
    sustained = None
    if args.sustained_steps > 0 and flush_buf is None:
        st2 = ctx.stats()
        ms_s, clocks_s = timed_rounds(torch, step, args.sustained_steps, barrier, local, None)
        ms_s = max_over_ranks(ms_s, world, dev)
        st3 = ctx.stats()
        kern_s, _ = stage_split(st2, st3, per_coord, d_local, peak, clocks_s.get("sm_mhz"))
        gbs_s = step_bytes / (ms_s * 1e-3) / 1e9
        sustained = {"steps": args.sustained_steps, "ms_per_step": ms_s, "sm_mhz": clocks_s.get("sm_mhz"),
                     "ms_x_mhz": ms_s * clocks_s["sm_mhz"] if clocks_s.get("sm_mhz") else None,
                     "reasons": clocks_s.get("reasons"), "value": (world if split == "none" else 1) * M * d * 4 / (ms_s * 1e-3) / 1e9,
                     "step_hbm": {"GBps": gbs_s, "frac_of_measured": gbs_s / peak, "frac_of_nominal_8TBps": gbs_s / NOMINAL_HBM_GBS},
                     "kernels": {k: {f: v[f] for f in ("ms", "kcycles", "frac_of_measured") if f in v} for k, v in kern_s.items()}}
        launches_note = int(st3.kernel_launches - st2.kernel_launches)
        sustained["gpu_launches"] = launches_note

    # ---- end to end: host buffers through tng_step_host, copies inside the timed region
    e2e = None
    if not args.no_e2e and split == "none":
        ctx_h = tng.Context(d, M, K, codec, norm, block=cfg["block"], fuse_mode=fuse, qsgd_levels=cfg.get("levels", 7),
                            host_staging=1, seed_lo=rank)
        for j in range(K):
            ctx_h.push_reference(ctx.history(K - 1 - j))
        g_host = torch.empty((M, d), dtype=torch.float32).pin_memory()
        g_host.copy_(batches[0])
        o_host = torch.empty(d, dtype=torch.float32).pin_memory()
        e2e_steps = max(1, min(args.steps, args.e2e_steps))
        for _ in range(2):
            ctx_h.step_host(g_host, o_host)
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            ctx_h.step_host(g_host, o_host)
        torch.cuda.synchronize()
        dt_blocking = max_over_ranks((time.perf_counter() - t0) / e2e_steps, world, dev)
        # the same rounds without waiting in between: the aggregate of round i travels to the host while
        # the rows of round i + 1 travel to the device; every copy still happens inside the timed region
        ctx_h.step_host_async(g_host, o_host)
        ctx_h.host_wait()
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            ctx_h.step_host_async(g_host, o_host)
        ctx_h.host_wait()
        torch.cuda.synchronize()
        dt = max_over_ranks((time.perf_counter() - t0) / e2e_steps, world, dev)
        e2e = {"value": job_throughput_gbs(world, M, d, dt), "unit": UNIT, "h2d_bytes_per_step": M * d * 4,
               "d2h_bytes_per_step": d * 4, "steps": e2e_steps, "ms_per_step": dt * 1e3,
               "api": "tng_step_host_async + tng_host_wait (pinned host rows -> device staging -> round -> aggregate back "
                      "to the host, the copy back overlapping the next round's rows)",
               "blocking": {"value": job_throughput_gbs(world, M, d, dt_blocking), "ms_per_step": dt_blocking * 1e3,
                            "api": "tng_step_host (returns when the aggregate is on the host)"}}
        ctx_h.close()
        del g_host, o_host

    line = None
    if rank == 0:
        # independent problems: every rank pushes its own M x d per round (weak); a split problem is ONE M x d problem (strong)
        value = job_throughput_gbs(world if split == "none" else 1, M, d, ms_step * 1e-3)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak" if split == "none" else "strong",
            "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": config_dict(name, cfg, world, split, flush_buf is not None), "clocks": clocks, "e2e": e2e,
            "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu_baseline,
            "coords_per_s": (world if split == "none" else 1) * M * d / (ms_step * 1e-3),
            "bits_per_coord": st1.bits_per_coord,
            "step_hbm": {"algorithmic_bytes_per_coord": sum(per_coord.values()), "GBps": step_gbs,
                         "frac_of_measured": step_gbs / peak, "frac_of_nominal_8TBps": step_gbs / NOMINAL_HBM_GBS,
                         "ms_x_mhz": ms_step * clocks["sm_mhz"] if clocks.get("sm_mhz") else None},
            "sustained": sustained,
            "kernels": kernels, "cnz": st1.cnz, "solver_fallback": int(st1.solver_fallback),
            "nonfinite_scales": int(st1.nonfinite_scales),
        }
        if split != "none":
            _, wire_words, _, wire_scales = ctx.wire_pointers()
            line["exchange_per_round"] = exchange_bytes(split, world, M, wire_words, wire_scales)
        if emit:
            print(json.dumps(line), flush=True)
    ctx.close()
    del batches, out, flush_buf
    torch.cuda.empty_cache()
    if launched and emit:
        dist.destroy_process_group()
    return line


def run_c4_sweep(args):
    """The codec sweep: d in 2^20 .. 2^28, 1/2/4-bit codes, difference and quotient form, sigma in {0.1, 1};
    M = 8, K = 8, AR(1) reference trajectory.  One JSON line per point; with --out a markdown table too."""
    rows = []
    ds = [1 << 20, 1 << 22, 1 << 24, 1 << 26, 1 << 28] if args.d is None else [args.d]
    for d in ds:
        for codec in ("sign1", "tern2", "qsgd4"):
            for norm in ("diff", "quot"):
                for sigma in (0.1, 1.0):
                    cfg = dict(WORKLOADS["c4_point"], d=d, codec=codec, norm=norm, sigma=sigma)
                    line = run_ours(args, f"c4_sweep d=2^{d.bit_length() - 1} {codec} {norm} sigma={sigma}", cfg, emit=False)
                    if line is None:
                        continue
                    point = {"workload": "c4_sweep", "d": d, "codec": codec, "norm": norm, "sigma": sigma, "M": 8, "K": 8,
                             "steps": args.steps, "ms_per_step": line["ms_per_step"], "value": line["value"], "unit": UNIT,
                             "frac_of_measured": line["step_hbm"]["frac_of_measured"],
                             "frac_of_nominal_8TBps": line["step_hbm"]["frac_of_nominal_8TBps"],
                             "bits_per_coord": line["bits_per_coord"], "cnz": line["cnz"], "l2": line["config"]["l2"][:10],
                             "sm_mhz": line["clocks"].get("sm_mhz"), "kernels_ms": {k: v["ms"] for k, v in line["kernels"].items()}}
                    print(json.dumps(point), flush=True)
                    rows.append(point)
    if args.out and rows:
        with open(args.out, "w") as f:
            f.write("| d | codec | form | sigma | ms/round | GB/s of gradient | of measured HBM | of 8 TB/s | bits/coord | C_nz |\n")
            f.write("|---|---|---|---|---|---|---|---|---|---|\n")
            for r in rows:
                f.write(f"| 2^{r['d'].bit_length() - 1} | {r['codec']} | {r['norm']} | {r['sigma']} | {r['ms_per_step']:.3f} | {r['value']:.0f} | "
                        f"{r['frac_of_measured']:.3f} | {r['frac_of_nominal_8TBps']:.3f} | {r['bits_per_coord']:.3f} | {r['cnz']:.4f} |\n")


def rank_check(args):
    """The launcher path without a GPU: the ranks meet over gloo, agree on the slowest rank's time and
    assemble a wire the way the worker split does.  Rank 0 prints one JSON line."""
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo")
    job_ms = max_over_ranks(1.0 + rank, world, "cpu")
    wire = torch.zeros((world, 4), dtype=torch.int32)
    wire[rank] = rank + 1
    if world > 1:
        dist.all_gather_into_tensor(wire, wire[rank:rank + 1].clone())
        dist.barrier()
    if rank == 0:
        print(json.dumps({"rank_check": True, "n_gpus": world, "job_ms": job_ms, "wire_rows": wire[:, 0].tolist()}), flush=True)
    if world > 1:
        dist.destroy_process_group()


def launch_command(n, argv, port):
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
            "--master-port", str(port), str(Path(__file__).resolve())] + list(argv)


def launch_ranks(n, argv):
    """Start n ranks of this script on this node (one per GPU) and wait for them: what
    `python -m torch.distributed.run --nnodes=1 --nproc-per-node n ... bench.py <argv>` does."""
    import socket
    import subprocess
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    env = dict(os.environ)
    # the communicator log lets a reader of the output count the ranks that really joined; keep it off stdout
    env.setdefault("NCCL_DEBUG", "INFO")
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    env.setdefault("NCCL_DEBUG_FILE", "/dev/stderr")
    return subprocess.call(launch_command(n, argv, port), env=env)


def run_producers(args):
    """Side benchmark (not the headline line): the local-gradient producers of the synthetic
    workloads, each against its own HBM roofline.  Logistic regression at the dense
    configuration's per-worker shape (n = 2048 samples x d = 65536 features; the gradient needs
    two passes over the 512 MiB of features: margins, then the transposed product) and the
    extended Rosenbrock gradient at d = 2^20, M = 32 (reads x and the M noise rows, writes M rows)."""
    import torch

    from paper_1901_08227_b200 import tng, workloads
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    peak, peak_src = measured_hbm_peak()
    steps, warm = (args.steps or 20), max(args.warmup or 3, 3)

    def timed(fn):
        for _ in range(warm):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps

    out = {}
    n, d = 2048, 65536
    X = workloads.normal((n, d), 0, 1, dev)
    b = torch.sign(workloads.normal((n,), 0, 2, dev))
    w = workloads.normal((d,), 0, 3, dev, std=0.01)
    grad = torch.empty(d, device=dev)
    scratch = torch.empty(tng.logistic_scratch_floats(n, d), device=dev)
    ms = timed(lambda: tng.logistic_grad(X, b, w, 1e-4, grad, scratch))
    by = 2.0 * n * d * 4
    out["logistic_grad"] = {"shape": f"n={n}, d={d}", "ms": ms, "algorithmic_bytes": by, "GBps": by / ms / 1e6,
                            "frac_of_measured": by / ms / 1e6 / peak}
    del X
    d3, M3 = 1 << 20, 32
    x = workloads.rosenbrock_x0(0, d3, dev)
    noise = workloads.rosenbrock_noise(0, 0, M3, d3, dev)
    g = torch.empty((M3, d3), device=dev)
    ms = timed(lambda: tng.rosenbrock_grad(x, noise, g))
    by = (2.0 * M3 + 1) * d3 * 4
    out["rosenbrock_grad"] = {"shape": f"d={d3}, M={M3}", "ms": ms, "algorithmic_bytes": by, "GBps": by / ms / 1e6,
                              "frac_of_measured": by / ms / 1e6 / peak,
                              "note": "256 MiB per launch: partly served by the 126 MB L2"}
    print(json.dumps({"workload": "producers", "peak_GBps": peak, "peak_source": peak_src, "steps": steps, "kernels": out}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c5_dnn_stream", choices=sorted(WORKLOADS) + ["producers", "c4_sweep"])
    ap.add_argument("--split", default="none", choices=["none", "workers", "coords"],
                    help="how several GPUs share the work: independent problems, the M workers spread over the ranks, "
                         "or the coordinates spread over the ranks (both also run on one GPU through the same rank-local calls)")
    ap.add_argument("--e2e-steps", type=int, default=8)
    ap.add_argument("--sustained-steps", type=int, default=None, help="rounds of the second, long timed region (0 = none)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--rank-check", action="store_true", help="CPU-only check of the launcher path (gloo)")
    ap.add_argument("--out", default=None, help="c4_sweep: also write the table as markdown to this file")
    # overrides for sweeps over the codec-sweep configuration (not the headline line)
    ap.add_argument("--d", type=int, default=None)
    ap.add_argument("--codec", choices=["sign1", "tern2", "qsgd4"], default=None)
    ap.add_argument("--norm", choices=["none", "diff", "quot", "comb", "mean"], default=None)
    ap.add_argument("--fuse", choices=["lsq", "last", "mean", "hindsight"], default=None)
    ap.add_argument("--block", type=int, default=None)
    ap.add_argument("--levels", type=int, default=None)
    args = ap.parse_args()
    # --gpus N without a launcher: start the N ranks here
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and (args.impl == "ours" or args.rank_check):
        sys.exit(launch_ranks(args.gpus, sys.argv[1:]))
    if args.rank_check:
        rank_check(args)
        return
    if args.workload == "producers":
        run_producers(args)
        return
    if args.workload == "c4_sweep":
        args.steps = 20 if args.steps is None else args.steps
        args.warmup = 3 if args.warmup is None else max(args.warmup, 3)
        args.no_e2e = args.no_cpu_baseline = True
        args.sustained_steps = 0
        run_c4_sweep(args)
        return
    cfg = dict(WORKLOADS[args.workload])
    for key in ("d", "codec", "norm", "fuse", "block", "levels"):
        if getattr(args, key) is not None:
            cfg[key] = getattr(args, key)
            args.workload = f"{args.workload}+{key}={cfg[key]}"
    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args, args.workload, cfg)
        return
    args.steps = 100 if args.steps is None else args.steps          # the stream configuration's own step count
    args.warmup = 5 if args.warmup is None else max(args.warmup, 3)  # never fewer than 3 warm-up rounds
    if args.sustained_steps is None:
        args.sustained_steps = 1000 if args.workload == "c5_dnn_stream" and args.split == "none" else 0
    run_ours(args, args.workload, cfg)


if __name__ == "__main__":
    main()
