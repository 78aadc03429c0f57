#!/usr/bin/env python
"""Benchmark of the straggler-scoring hot path on B200.

One "step" is one pass of the whole path over the large-fleet workload: 16 384 ranks x
20 000 steps x 8 float32 metrics (10.49 GB), ingested in 100 blocks of 200 steps with one
evaluation (windowed medians, fleet baseline, scores/flags/tiers, top-64) after each block.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line.  `value` is cells scored per second with the telemetry already
resident in HBM (written in place into the library's ring before the timed region);
`e2e` is the same metric with the telemetry in pinned HOST memory, copied block by block
into the ring inside the timed region (on a copy stream, one block ahead of the scoring),
and the flags / top-k of every evaluation read back to the host.  With N > 1 every rank runs an independent replica (the path does not
shard: a cross-rank median needs all ranks of a step on one GPU).

`--impl reference` times the CPU oracle (oracle/, single thread, as it stands) on a
bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "rank-step-metric cells scored/s"
UNIT = "cells/s"
L2_BYTES = 126 * 1024 * 1024
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel on this workload, from
# the ncu capture summarised under profiles/ (None once the kernel has changed since the capture)
NCU_TRAFFIC_BYTES_PER_LAUNCH = 112.0e6   # window_thread_kernel 110.72e6 + its finishing kernel (~200 series x 6.4 KB)
# which kernel the roofline object describes: 2 = window_thread_kernel (guard_score), 1 = the MAD sweep (guard_ingest)
PROFILE_MODE = 2
PROFILE_KERNEL = ("window_thread_kernel + window_finish_kernel (windowed per-rank medians of one evaluation)" if PROFILE_MODE == 2 else
                  "xsplit_sweep_kernel<2,1> (cross-rank MAD / exceedance sweep of one ingested block)")
FALLBACK_HBM_GBS = 6650.0   # earlier measurement on this machine, used only if MEASURED_PEAKS.json is absent


def measured_hbm_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self, t_begin=None, t_end=None):
        """Summary of the samples taken between the host times t_begin and t_end (the timed region);
        if the region was too short to catch one, of the samples within half a second around it."""
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        try:
            self.proc.terminate()
            self.proc.wait(timeout=5)
        except Exception:
            pass
        recs = []
        try:
            for ln in open(self.path):
                p = [x.strip() for x in ln.split(",")]
                if len(p) < 9:
                    continue
                try:
                    ts = datetime.datetime.strptime(p[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    recs.append((ts, float(p[1]), float(p[2]), p[5:9]))
                except ValueError:
                    continue
            os.unlink(self.path)
        except Exception:
            pass
        window = "timed region"
        sel = recs
        if t_begin is not None and t_end is not None:
            sel = [r for r in recs if t_begin <= r[0] <= t_end]
            if not sel:
                sel = [r for r in recs if t_begin - 0.5 <= r[0] <= t_end + 0.5]
                window = "within 0.5 s of the timed region (the same load: warm-up passes run right before it)"
        reasons = set()
        for r in sel:
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if sel:
            out.update(sm_mhz=statistics.median([r[1] for r in sel]), sm_max_mhz=max(r[2] for r in sel), samples=len(sel),
                       window=window)
        out["reasons"] = sorted(reasons)
        return out


def workload():
    from paper_2605_17879_b200 import synth
    return synth.paper_configs()["large"]


def oracle_sample_rate(cfg, block_host, sample_steps):
    """Cells per second of the CPU oracle on the first `sample_steps` steps of one block
    (ingest + one evaluation), single thread."""
    from oracle import guard_oracle as go
    from paper_2605_17879_b200 import synth
    o = go.Oracle(cfg.ranks, cfg.metrics, cfg.W, cfg.k, cfg.topk, dir=synth.fleet_dir(cfg.metrics))
    x = block_host[:sample_steps]
    t0 = time.perf_counter()
    o.ingest(x)
    o.score()
    dt = time.perf_counter() - t0
    return x.size / dt, dt


def _oracle_block_worker(job):
    """One 200-step block of the workload through the oracle (as it stands, one thread): generated on the
    CPU by the same seeded generator, then ingest + one evaluation are timed.  Runs in a spawned process."""
    t0_step, = job
    import torch
    torch.set_num_threads(1)
    from oracle import guard_oracle as go
    from paper_2605_17879_b200 import synth
    cfg = synth.paper_configs()["large"]
    blk = synth.fleet_block(cfg, t0_step, t0_step + cfg.block, device="cpu").numpy()
    o = go.Oracle(cfg.ranks, cfg.metrics, cfg.W, cfg.k, cfg.topk, dir=synth.fleet_dir(cfg.metrics))
    t0 = time.perf_counter()
    o.ingest(blk)
    o.score()
    return blk.size, time.perf_counter() - t0


def oracle_all_cores(cfg):
    """The oracle on all host cores: the workload's outermost independent loop (its 200-step blocks: windows are
    tumbling, so blocks do not depend on one another) split over one spawned process per core, one block
    each.  The oracle's source is untouched.  Returns the cpu_baseline sub-object."""
    import multiprocessing as mp
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    workers = max(1, min(cores, cfg.steps // cfg.block, 32))
    model = "unknown"
    try:
        for ln in open("/proc/cpuinfo"):
            if ln.startswith("model name"):
                model = ln.split(":", 1)[1].strip()
                break
    except Exception:
        pass
    ctx = mp.get_context("spawn")
    wall0 = time.perf_counter()
    with ctx.Pool(workers) as pool:
        res = pool.map(_oracle_block_worker, [(j * cfg.block,) for j in range(workers)])
    wall = time.perf_counter() - wall0
    cells = sum(r[0] for r in res)
    slowest = max(r[1] for r in res)
    return {"value": cells / slowest, "unit": UNIT, "cores": workers, "host_cores": cores, "cpu_model": model, "kind": "oracle",
            "seconds": slowest, "wall_seconds_with_generation": wall,
            "sample": "%d blocks of 200 steps at full width, one per spawned process, each ingest + one evaluation; "
                      "rate = cells of all blocks / slowest process" % workers}


def run_sweep(dev, reps=10):
    """Offline node-sweep qualification (2 048 nodes x 8 GPUs x 200 repetitions x 6 metrics, 78.6 MB), timed with
    CUDA events; algorithmic traffic is one 4-byte read per cell."""
    import torch
    from paper_2605_17879_b200 import guard, synth
    cfg = synth.SweepConfig()
    S = synth.sweep_tensor(cfg, device=dev)
    kw = dict(dir=synth.sweep_dir(cfg.metrics), thr=3.5, floor_rel=1e-4, floor_abs=synth.sweep_floor_abs(cfg.metrics),
              pct_ppm=cfg.pct_ppm)
    out = guard.sweep_qualify(S, cfg.nodes, cfg.gpus_per_node, **kw)
    ws = torch.empty(int(guard.lib().guard_sweep_workspace_bytes(cfg.gpus, cfg.reps, cfg.metrics)), dtype=torch.uint8, device=dev)
    flush = torch.empty(L2_BYTES * 2, dtype=torch.uint8, device=dev)
    times = []
    for _ in range(3 + reps):
        flush.zero_()                                # the 78.6 MB input would otherwise sit in L2 between repetitions
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        guard.sweep_qualify(S, cfg.nodes, cfg.gpus_per_node, workspace=ws, out=out, **kw)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) / 1e3)
    t = statistics.median(times[3:])
    peak, _ = measured_hbm_peak()
    cells = S.numel()
    return {"workload": "node sweep: %d nodes x %d GPUs x %d repetitions x %d metrics (%.1f MB), L2 flushed between repetitions"
                        % (cfg.nodes, cfg.gpus_per_node, cfg.reps, cfg.metrics, cells * 4 / 1e6),
            "ms": t * 1e3, "cells_per_s": cells / t, "algorithmic_GBps": cells * 4 / t / 1e9,
            "frac_of_peak": cells * 4 / t / 1e9 / peak, "gpus_failed": int((out["gpu_pass"] == 0).sum().item()),
            "status": int(out["status"].item())}


def run_small_config(dev, name, passes=5):
    """Whole-path throughput of one of the smaller fleet configurations (resident telemetry, deferred mode)."""
    import torch
    from paper_2605_17879_b200 import guard, synth
    cfg = synth.paper_configs()[name]
    R, M, T, B = cfg.ranks, cfg.metrics, cfg.steps, cfg.block
    g = guard.Guard(R, M, cfg.W, cfg.k, dir=synth.fleet_dir(M), capacity=T, topk=cfg.topk, device=dev)
    ring = g.ring_reserve(T)
    ring.copy_(synth.fleet_tensor(cfg, device=dev))
    out = g.alloc_outputs()
    g.set_deferred(True)

    def one_pass():
        g.reset()
        for j in range(T // B):
            g.ingest(ring[j * B:(j + 1) * B])
            g.score(out)
        g.join()

    for _ in range(2):
        one_pass()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(passes):
        one_pass()
    e1.record()
    torch.cuda.synchronize()
    g.sync_status()
    secs = e0.elapsed_time(e1) / 1e3 / passes
    g.close()
    return {"workload": "%s fleet: %d ranks x %d steps x %d metrics, W=%d, blocks of %d (launch-bound at this size)"
                        % (name, R, T, M, cfg.W, B), "ms_per_pass": secs * 1e3, "cells_per_s": R * M * T / secs}


def run_streaming(dev, steps, warm):
    """Streaming configuration: 32 768 ranks x 8 metrics, one step per ingest into a 512-step
    ring, an evaluation after every step, flags and top-k read back to pinned host memory.
    Latency leg: the step is landed in its ring slot before the clock starts (in-place ingest).
    Sustained leg: guard_ingest copies each step from a staging buffer into the ring (one call
    per step), deferred evaluations, joined before the clock stops.
    Returns per-step ingest-to-flag latency percentiles (host clock) and sustained cells/s."""
    import torch
    from paper_2605_17879_b200 import guard, synth
    cfg = synth.paper_configs()["streaming"]
    R, M = cfg.ranks, cfg.metrics
    g = guard.Guard(R, M, cfg.W, cfg.k, dir=synth.fleet_dir(M), capacity=cfg.ring_capacity, topk=cfg.topk, device=dev)
    pool = 256                                   # generated steps, produced outside the timed region
    gen = synth.fleet_block(cfg, 0, pool, device=dev)
    out = g.alloc_outputs()
    h_flags = torch.empty(R, dtype=torch.uint8, pin_memory=True)
    h_idx = torch.empty(cfg.topk, dtype=torch.int32, pin_memory=True)
    lat = []

    def one(t, timed):
        slot = g.ring_reserve(1)
        slot.copy_(gen[t % pool:t % pool + 1])    # the producer lands the step in its ring slot
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        g.ingest(slot)
        g.score(out)
        h_flags.copy_(out["flags"], non_blocking=True)
        h_idx.copy_(out["topk_idx"], non_blocking=True)
        torch.cuda.synchronize()
        if timed:
            lat.append(time.perf_counter() - t0)

    for t in range(warm):
        one(t, False)
    for t in range(warm, warm + steps):
        one(t, True)
    # sustained: no host synchronisation between steps, deferred evaluations (an evaluation runs
    # beside the next step's ingest), joined before the clock stops
    torch.cuda.synchronize()
    g.set_deferred(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    src = [gen[i:i + 1] for i in range(pool)]    # the producer's staging buffers: guard_ingest copies a step into the ring
    e0.record()
    for t in range(steps):
        g.ingest(src[t % pool])
        g.score(out)
    g.join()
    e1.record()
    torch.cuda.synchronize()
    g.sync_status()
    sustained = steps * R * M / (e0.elapsed_time(e1) / 1e3)
    lat.sort()
    pick = lambda q: lat[min(len(lat) - 1, int(q * len(lat)))] * 1e6
    res = {"workload": "streaming: 32768 ranks x 8 metrics, ring 512, W=200 k=120 top-64, evaluation every step",
           "steps": steps, "latency_us": {"p50": pick(0.50), "p99": pick(0.99), "max": lat[-1] * 1e6},
           "sustained_cells_per_s": sustained, "us_per_step_sustained": e0.elapsed_time(e1) * 1e3 / steps,
           "cells_per_step": R * M, "fallback_rows": g.fallback_steps(),
           "sliding_rebuilds_per_step": g.sliding_rebuilds() / float(warm + 2 * steps)}
    g.close()
    return res


def run_reference(args):
    """The reference arm: the oracle as it stands, on the host cores."""
    from paper_2605_17879_b200 import dist as gd, synth
    rank, _, world = gd.env_world()
    if rank != 0:
        return 0
    cfg = workload()
    sample_steps = 40
    block = synth.fleet_block(cfg, 0, sample_steps, device="cpu").numpy()
    from oracle import guard_oracle as go
    go.build()
    for _ in range(max(0, min(args.warmup, 1))):
        oracle_sample_rate(cfg, block, 8)
    times = []
    for _ in range(args.steps):
        rate, dt = oracle_sample_rate(cfg, block, sample_steps)
        times.append(dt)
    total = sum(times)
    cells = block.size * args.steps
    value = cells / total
    sample = ("per step: ingest + one evaluation of the first %d steps of the workload at full width "
              "(%d ranks x %d metrics), window = those %d steps" % (sample_steps, cfg.ranks, cfg.metrics, sample_steps))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "large fleet: 16384 ranks x 20000 steps x 8 metrics, W=200 k=120 top-64 (bounded sample)"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="guard", choices=["guard", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-all-cores", action="store_true", help="skip the all-core leg of the CPU baseline")
    ap.add_argument("--streaming-steps", type=int, default=500)
    ap.add_argument("--only", default="", choices=["", "streaming", "sweep"],
                    help="run only this secondary leg and print its object (for profiling; not a bench line)")
    ap.add_argument("--blocks", type=int, default=0,
                    help="profile-sized run: only this many 200-step blocks of the workload (0 = all 100); not a bench value")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.only:
        # profile-sized runs of one secondary leg (not a bench line): prints that leg's object only
        import torch
        from paper_2605_17879_b200 import guard
        guard.lib()
        dev = torch.device("cuda", 0)
        torch.cuda.set_device(dev)
        res = run_streaming(dev, args.streaming_steps, 250) if args.only == "streaming" else run_sweep(dev)
        print(json.dumps({"only": args.only, "result": res}), flush=True)
        return 0

    import torch
    from paper_2605_17879_b200 import dist as gd, guard, synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    guard.lib()   # fails loudly if the CUDA library is not built
    rank, local_rank, world = gd.init("nccl")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    warm = max(3, args.warmup)

    cfg = workload()
    if args.blocks > 0:
        import dataclasses
        cfg = dataclasses.replace(cfg, steps=max(2, args.blocks) * cfg.block)
    R, M, T, B = cfg.ranks, cfg.metrics, cfg.steps, cfg.block
    n_blocks = T // B
    dirs = synth.fleet_dir(M)
    # the ring holds the whole tensor, so telemetry is written in place once and stays resident
    g = guard.Guard(R, M, cfg.W, cfg.k, dir=dirs, capacity=T, topk=cfg.topk, device=dev)
    ring = g.ring_reserve(T)
    for t0 in range(0, T, B):
        synth.fleet_block(cfg, t0, t0 + B, device=dev, out=ring[t0:t0 + B])
    torch.cuda.synchronize()
    out = g.alloc_outputs()
    cells_per_step = R * M * T

    # Deferred evaluations: an evaluation runs beside the next block's ingest; its outputs are
    # complete once the stream has passed the next score() or join().  Every pass ends with a join.
    g.set_deferred(True)

    def one_pass():
        g.reset()
        for j in range(n_blocks):
            g.ingest(ring[j * B:(j + 1) * B])
            g.score(out)
        g.join()

    sampler = ClockSampler(local_rank)
    sampler.start()   # nvidia-smi needs a moment before its first sample: started ahead of the warm-up passes
    for _ in range(warm):
        one_pass()
    g.sync_status()
    g.profile_enable(PROFILE_MODE)
    launches0 = g.kernel_launches
    gd.barrier()
    torch.cuda.synchronize()
    t_begin = time.time()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(args.steps):
        one_pass()
    stop.record()
    torch.cuda.synchronize()
    t_end = time.time()
    gd.barrier()
    clocks = sampler.stop(t_begin, t_end)
    kern_ms, kern_n = g.profile_read()
    g.profile_enable(False)
    g.sync_status()
    launches = g.kernel_launches - launches0
    fallback_rows = g.fallback_steps()
    secs = start.elapsed_time(stop) / 1e3
    value, tmax = gd.aggregate_throughput(cells_per_step * args.steps, secs, device=dev)
    flagged = int(out["flags"].sum().item())

    # roofline of the dominant kernel, timed by the library with CUDA events recorded right around
    # it on the stream it is launched on (while the other kernels of the pipeline share the GPU).
    # The window-median kernel reads the W x ranks x metrics window once (4 B per cell covered);
    # the MAD / exceedance sweep reads a block of 200 steps once (4 B per cell) and writes one
    # exceedance byte per (step, rank).
    launch_s = (kern_ms / kern_n / 1e3) if kern_n else float("nan")
    algo_bytes = (cfg.W * R * M * 4) if PROFILE_MODE == 2 else (B * R * M * 4 + B * R * 1)
    peak, peak_kind = measured_hbm_peak()
    achieved = algo_bytes / launch_s / 1e9
    roofline = {"bound": "hbm", "kernel": PROFILE_KERNEL,
                "achieved": achieved, "peak": peak, "peak_source": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH, "algorithmic_bytes_per_launch": algo_bytes,
                "avg_launch_ms": launch_s * 1e3, "launches_timed": kern_n,
                "share_of_step": (kern_ms / 1e3 / secs) if kern_n else None,
                "path_algorithmic_GBps": (8.125 * cells_per_step * args.steps) / secs / 1e9,
                "path_frac_of_peak": (8.125 * cells_per_step * args.steps) / secs / 1e9 / peak}

    # end to end: telemetry in pinned host memory, copied into the ring block by block,
    # flags and top-k copied back after every evaluation
    need_host = args.e2e_steps > 0 or (rank == 0 and world == 1 and not args.no_cpu_baseline)
    host = torch.empty((T if args.e2e_steps > 0 else B, R, M), dtype=torch.float32, pin_memory=True) if need_host else None
    if need_host:
        host.copy_(ring[:host.shape[0]])
    h_flags = torch.empty(R, dtype=torch.uint8, pin_memory=True)
    h_idx = torch.empty(cfg.topk, dtype=torch.int32, pin_memory=True)
    h_sc = torch.empty(cfg.topk, dtype=torch.float32, pin_memory=True)
    torch.cuda.synchronize()

    # End to end: block j + 1 is copied from pinned host memory on a copy stream while block j is
    # ingested and evaluated (deferred mode); the flags and top-k of every evaluation are read back to
    # the host as soon as that evaluation has been joined (by the next score(), or the final join()).
    copy_stream = torch.cuda.Stream(device=dev)
    copied = [torch.cuda.Event() for _ in range(n_blocks)]
    outs2 = [out, g.alloc_outputs()]

    def read_back(o):
        h_flags.copy_(o["flags"], non_blocking=True)
        h_idx.copy_(o["topk_idx"], non_blocking=True)
        h_sc.copy_(o["topk_score"], non_blocking=True)

    def one_pass_e2e():
        g.reset()
        main = torch.cuda.current_stream()
        copy_stream.wait_stream(main)   # the ring is free again: everything of the previous pass has been joined
        with torch.cuda.stream(copy_stream):
            for j in range(n_blocks):
                ring[j * B:(j + 1) * B].copy_(host[j * B:(j + 1) * B], non_blocking=True)
                copied[j].record(copy_stream)
        for j in range(n_blocks):
            main.wait_event(copied[j])
            g.ingest(ring[j * B:(j + 1) * B])
            g.score(outs2[j % 2])       # joins evaluation j - 1
            if j > 0:
                read_back(outs2[(j - 1) % 2])
        g.join()
        read_back(outs2[(n_blocks - 1) % 2])

    e2e = None
    if args.e2e_steps > 0:
        one_pass_e2e()
        gd.barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            one_pass_e2e()
        torch.cuda.synchronize()
        e2e_secs = time.perf_counter() - t0
        gd.barrier()
        e2e_value, _ = gd.aggregate_throughput(cells_per_step * args.e2e_steps, e2e_secs, device=dev)
        e2e = {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": T * R * M * 4,
               "d2h_bytes_per_step": n_blocks * (R + 8 * cfg.topk), "steps": args.e2e_steps,
               "ms_per_step": 1e3 * e2e_secs / args.e2e_steps}
    g.sync_status()

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sample_steps = B          # one whole block with its full window: the unit the workload repeats
        blk = host[:sample_steps].numpy()
        rate, dt = oracle_sample_rate(cfg, blk, sample_steps)
        cpu_baseline = {"value": rate, "unit": UNIT, "cores": 1, "kind": "oracle", "seconds": dt,
                        "sample": "ingest + one evaluation of the first %d steps at full width (%d ranks x %d metrics)"
                                  % (sample_steps, R, M)}
        if not args.no_all_cores:
            cpu_baseline["all_cores"] = oracle_all_cores(cfg)

    streaming = None
    other = None
    if rank == 0 and world == 1 and args.streaming_steps > 0:
        del ring, out
        g.close()
        torch.cuda.empty_cache()
        # 250 warm-up steps: the 200-step window is full and the sliding state settled before anything is timed
        streaming = run_streaming(dev, args.streaming_steps, 250)
        other = {"sweep": run_sweep(dev), "tiny": run_small_config(dev, "tiny"), "medium": run_small_config(dev, "medium")}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warm,
            "ms_per_step": 1e3 * tmax / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": ("large fleet: 16384 ranks x 20000 steps x 8 metrics (10.49 GB), W=200 k=120 top-64, "
                                    "100 blocks of 200 steps, one evaluation per block") if args.blocks <= 0 else
                                   ("PROFILE-SIZED RUN (not a bench value): %d blocks of the large fleet" % (T // B)),
                       "ingest": "in place (telemetry written into the ring before timing)",
                       "evaluation": "deferred (guard_set_deferred): each evaluation runs beside the next block's ingest, "
                                     "joined before its outputs are reused and at the end of every pass",
                       "l2": "inputs (10.49 GB) larger than L2", "parallelism": "replicas only",
                       "flagged_last_evaluation": flagged, "direct_path_fallback_rows_last_pass": fallback_rows},
            "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": launches, "clocks": clocks,
            "streaming": streaming, "other_configs": other,
        }
        print(json.dumps(line), flush=True)
    g.close()
    gd.finish()
    return 0


if __name__ == "__main__":
    sys.exit(main())
