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
    # name: d, M, K, norm, codec, block
    "c5_dnn_stream": dict(d=1 << 27, M=8, K=8, norm="quot", codec="tern2", block=128, fuse="lsq"),
    "c5_mid": dict(d=1 << 24, M=8, K=8, norm="quot", codec="tern2", block=128, fuse="lsq"),   # profiler-sized
    "c5_small": dict(d=1 << 22, M=8, K=8, norm="quot", codec="tern2", block=128, fuse="lsq"),
}


def algorithmic_bytes_per_coord(M, K, bits, block, fuse, user_out=True, ref_in_encode=True, norm="quot"):
    """Bytes per coordinate each kernel of one round has to move (reads + writes).

    dots    reads the K ring rows and the M gradient rows;
    encode  reads the M gradient rows and writes the wire (codes + scales); with the reference
            combine folded into it (block 128) it also reads the K ring rows and writes the
            reference, otherwise it reads the reference a separate combine pass wrote;
    decode  reads the wire and the reference, writes the new ring entry (and the caller's copy).
    The combined form carries a second reference wherever the first one is read or written; the
    scalar reference has no fusion at all, its encode reads the gradient rows twice (means, then codes)."""
    wire = M * bits / 8.0 + 4.0 * M / block
    per = {}
    if norm == "mean":
        per["encode"] = 8.0 * M + wire
        per["decode"] = wire + 4.0 + (4.0 if user_out else 0.0)
        return per
    refs = 8.0 if norm == "comb" else 4.0
    if fuse == "lsq":
        per["dots"] = 4.0 * K + 4.0 * M
    elif fuse == "hindsight":
        per["dots"] = 4.0 * K                      # Gram of the ring only
    combines = fuse != "last"                      # the delayed-gradient reference is a ring slot as it is
    if combines and ref_in_encode:
        per["encode"] = 4.0 * K + 4.0 * M + refs + wire
    else:
        if combines:
            per["combine"] = 4.0 * K + refs
        per["encode"] = 4.0 * M + refs + wire
    per["decode"] = wire + refs + 4.0 + (4.0 if user_out else 0.0)
    return per


# dram__bytes_read.sum + dram__bytes_write.sum per coordinate of the dominant kernel, from the ncu
# capture summarised under profiles/ (taken at d = 2^24 and scaled by d: every kernel streams each
# coordinate once).  None = the kernel changed after the capture.
# integer/logic-pipe instructions the staged encode kernel issues per tile and worker (ternary, quotient
# form; from the opcode histogram of the same capture: 22 logic ops, 9 float compares, 8 ballots, 6 integer
# compares, 4 conversions, 3 integer adds, 3 max, 2 selects, 3 others)
ALU_PIPE_INSTR_PER_TILE_WORKER = 60
NCU_TRAFFIC_BYTES_PER_COORD = {"encode": 69.94, "dots": 64.25, "decode": 11.32}


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


def config_dict(name, cfg, world):
    return {"workload": name, "d": cfg["d"], "M": cfg["M"], "K": cfg["K"], "normalisation": cfg["norm"],
            "codec": cfg["codec"], "block": cfg["block"], "fusion": cfg["fuse"],
            "stream": "Student-t(nu=3) around an AR(1) mean (rho 0.99), 64 segments with LogUniform(1e-4,1e-1) scales",
            "l2": "inputs exceed L2: every round streams the whole ring and all M gradient rows from HBM",
            "sharding": "one process per GPU, each rank an independent problem of the full size (no data-path collective)" if world > 1 else "single GPU"}


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
    orc = oracle.State(d_s, M, K, codec, norm, block=cfg["block"], fuse_mode=fuse)
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
    orc = oracle.State(d_s, M, K, codec, norm, block=cfg["block"], fuse_mode=fuse)
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
           "sample": f"first {d_s} of {cfg['d']} coordinates per step, {n} steps, {per * 1e3:.1f} ms each"}
    if single_thread and cores > 1:
        # the same oracle on one thread, on a shorter sample (a quarter of the coordinates, one step)
        d_1 = max(d_s // 4, 1 << 14)
        orc1 = oracle.State(d_1, M, K, codec, norm, block=cfg["block"], fuse_mode=fuse)
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
def run_ours(args, name, cfg):
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
    if launched:
        dist.init_process_group("nccl", device_id=dev)
    tng.lib()                                       # fail loudly if libtng.so is missing

    norm, codec, fuse = enum_of(tng, cfg)
    d, M, K = cfg["d"], cfg["M"], cfg["K"]
    bits = codec

    cpu_baseline = None
    if rank == 0 and not args.no_cpu_baseline:
        cpu_baseline = time_cpu_baseline(cfg, (norm, codec, fuse))

    # ---- inputs, resident in HBM: ring pre-filled with K past means, two gradient batches
    stream = workloads.GradientStream(rank, d, M, device=dev)
    ctx = tng.Context(d, M, K, codec, norm, block=cfg["block"], fuse_mode=fuse, timing=1, seed_lo=rank)
    for _ in range(K):
        ctx.push_reference(stream.advance())
    batches = []
    for _ in range(2):
        stream.advance()
        batches.append(stream.worker_grads())
    out = torch.empty(d, device=dev)
    del stream
    torch.cuda.empty_cache()

    def barrier():
        if launched:
            dist.barrier()
        torch.cuda.synchronize()

    for w in range(args.warmup):
        ctx.step(batches[w % 2], out)
    barrier()
    st0 = ctx.stats()
    sampler = ClockSampler(local)
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for s in range(args.steps):
        ctx.step(batches[s % 2], out)
    ev1.record()
    barrier()
    clocks = sampler.stop()
    ms_step = max_over_ranks(ev0.elapsed_time(ev1), world, dev) / args.steps
    st1 = ctx.stats()
    launches = st1.kernel_launches - st0.kernel_launches

    # ---- per-kernel durations over the timed rounds (CUDA events recorded by the library on the same stream)
    n0, n1 = st0.timed_rounds, st1.timed_rounds
    def stage_ms(field):
        return (getattr(st1, field) * n1 - getattr(st0, field) * n0) / max(n1 - n0, 1)
    ref_in_encode = cfg["block"] == 128 and cfg["norm"] not in ("none", "mean") and stage_ms("ms_combine") == 0.0
    per_coord = algorithmic_bytes_per_coord(M, K, bits, cfg["block"], cfg["fuse"], ref_in_encode=ref_in_encode, norm=cfg["norm"])
    peak, peak_src = measured_hbm_peak()
    kernels = {}
    for kname, field in (("dots", "ms_dots"), ("combine", "ms_combine"), ("encode", "ms_encode"), ("decode", "ms_decode")):
        if kname not in per_coord:
            continue
        ms = stage_ms(field)
        gbs = per_coord[kname] * d / (ms * 1e-3) / 1e9 if ms > 0 else None
        kernels[kname] = {"ms": ms, "bytes_per_coord": per_coord[kname], "GBps": gbs, "frac_of_measured": gbs / peak if gbs else None}
    if ref_in_encode and "encode" in kernels:
        kernels["encode"]["includes"] = "reference combine (ring rows -> reference) folded into the encode pass"
    kernels["solve"] = {"ms": stage_ms("ms_solve")}
    dominant = max((k for k in kernels if "bytes_per_coord" in kernels[k]), key=lambda k: kernels[k]["ms"])
    # the counters were taken on the headline configuration; any other one has no capture
    profiled = all(cfg[k] == WORKLOADS["c5_dnn_stream"][k] for k in ("M", "K", "norm", "codec", "block", "fuse"))
    tpc = NCU_TRAFFIC_BYTES_PER_COORD.get(dominant) if profiled else None
    traffic = tpc * d if tpc is not None else None
    roofline = {"bound": "hbm", "kernel": dominant, "achieved": kernels[dominant]["GBps"], "peak": peak, "unit": "GB/s",
                "frac": kernels[dominant]["frac_of_measured"], "peak_source": peak_src, "traffic": traffic,
                "algorithmic_bytes_per_launch": per_coord[dominant] * d}
    if profiled and dominant == "encode" and clocks.get("sm_mhz"):
        # The encode pass is the one kernel that is closer to an arithmetic roof than to HBM: its busiest unit
        # is the integer/logic pipe, which takes one warp instruction every two cycles per SM partition
        # (4 partitions x 148 SMs).  The opcode histogram of the ncu capture gives about 60 such
        # instructions per tile (128 coordinates) and worker; stated beside the HBM figure, not instead of it.
        alu_peak = 0.5 * 4 * 148 * clocks["sm_mhz"] * 1e6
        alu_rate = ALU_PIPE_INSTR_PER_TILE_WORKER * (d / 128.0) * M / (kernels["encode"]["ms"] * 1e-3)
        roofline["alu_pipe"] = {"bound": "alu", "achieved": alu_rate / 1e9, "peak": alu_peak / 1e9, "unit": "G warp-instr/s",
                                "frac": alu_rate / alu_peak,
                                "peak_source": "0.5 warp-instr/cycle x 4 partitions x 148 SMs x sampled SM clock"}
    step_bytes = sum(per_coord.values()) * d
    step_gbs = step_bytes / (ms_step * 1e-3) / 1e9

    # ---- end to end: host buffers through tng_step_host, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        ctx_h = tng.Context(d, M, K, codec, norm, block=cfg["block"], fuse_mode=fuse, host_staging=1, seed_lo=rank)
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

    if rank == 0:
        value = job_throughput_gbs(world, M, d, ms_step * 1e-3)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": config_dict(name, cfg, world), "clocks": clocks, "e2e": e2e,
            "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu_baseline,
            "coords_per_s": world * M * d / (ms_step * 1e-3),
            "bits_per_coord": st1.bits_per_coord,
            "step_hbm": {"algorithmic_bytes_per_coord": sum(per_coord.values()), "GBps": step_gbs,
                         "frac_of_measured": step_gbs / peak, "frac_of_nominal_8TBps": step_gbs / NOMINAL_HBM_GBS},
            "kernels": kernels, "cnz": st1.cnz, "solver_fallback": int(st1.solver_fallback),
            "nonfinite_scales": int(st1.nonfinite_scales),
        }
        print(json.dumps(line), flush=True)
    ctx.close()
    if launched:
        dist.destroy_process_group()


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
    ap.add_argument("--workload", default="c5_dnn_stream", choices=sorted(WORKLOADS) + ["producers"])
    ap.add_argument("--e2e-steps", type=int, default=8)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    # overrides for sweeps over the codec-sweep configuration (not the headline line)
    ap.add_argument("--d", type=int, default=None)
    ap.add_argument("--codec", choices=["sign1", "tern2", "qsgd4"], default=None)
    ap.add_argument("--norm", choices=["none", "diff", "quot", "comb", "mean"], default=None)
    ap.add_argument("--fuse", choices=["lsq", "last", "mean", "hindsight"], default=None)
    args = ap.parse_args()
    if args.workload == "producers":
        run_producers(args)
        return
    cfg = dict(WORKLOADS[args.workload])
    for key in ("d", "codec", "norm", "fuse"):
        if getattr(args, key) is not None:
            cfg[key] = getattr(args, key)
            args.workload = f"{args.workload}+{key}={cfg[key]}"
    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args, args.workload, cfg)
        return
    args.steps = 200 if args.steps is None else args.steps
    args.warmup = 5 if args.warmup is None else max(args.warmup, 0)
    run_ours(args, args.workload, cfg)


if __name__ == "__main__":
    main()
