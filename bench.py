#!/usr/bin/env python
"""Throughput of batched exact lookup at 1,048,576 x 1024 bf16 centroids (queries per second).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--rows N --queries B]

A step is one lookup of a batch of 8,192 synthetic queries (top-4 + per-query hit threshold)
against the device-resident centroid matrix through the C ABI.  `value` times the call with the
batch already in HBM; `e2e` times the host-buffer entry point (pinned host memory in, results
back out).  With N > 1 (torchrun) every rank holds a replica of the cache and looks up its own
batch: weak scaling, no collective on the data path.  `--impl reference` times the CPU oracle
on a bounded sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "lookup queries/sec at 1Mx1024 bf16 centroids"
UNIT = "queries/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--rows", type=int, default=1 << 20, help="cached centroids (default: the full 1,048,576)")
    ap.add_argument("--queries", type=int, default=8192, help="query batch per step")
    ap.add_argument("--path", default="auto", choices=["auto", "simt", "tensor", "stream"])
    ap.add_argument("--workload", default="config4",
                    choices=["config4", "config1", "config2", "config3", "config5", "stream_probe", "cluster", "evict", "f32_lookup", "config5_full", "tiered"],
                    help="config4 (default) is the benchmark contract; the others print one line each for the other "
                         "configurations (single GPU only)")
    ap.add_argument("--dtype", default="f32", choices=["f32", "bf16"], help="vector type of the cluster workload")
    ap.add_argument("--seed", type=int, default=0, help="seed of the configuration-5 stream (config5_full)")
    ap.add_argument("--theta-range", type=float, nargs=2, default=None, metavar=("LO", "HI"),
                    help="config5_full: per-query thresholds uniform in [LO, HI] instead of the fixed 0.86")
    ap.add_argument("--maintain", action="store_true",
                    help="config5_full: after every million queries a MergeCentroids pass (theta_C 0.86, weighted mean) and the "
                         "decay of FilteringCentroids, as the paper re-clusters when enough new queries have arrived")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--sharded", action="store_true",
                    help="time the CENTROID-SHARDED cache instead of replicas: the rows of the workload are partitioned over the "
                         "--gpus ranks, every rank scores the same query batch against its rows, one all-gather of packed keys "
                         "(strong scaling); also times the sharded streaming step on the configuration-5 cache")
    ap.add_argument("--no-secondary", action="store_true",
                    help="skip the extra measurements of the default line (streaming step, small-batch sweeps, hit update)")
    return ap.parse_args()


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def workload(args, rank: int, threads: int):
    from gen import workloads as W
    n_clusters = max(64, args.rows // 16)
    return W.config(4, seed=0, query_seed=rank, mode="T", threads=threads, n_centroids=args.rows,
                    n_queries=args.queries, n_clusters=n_clusters)


def workload_name(args) -> str:
    return (f"config 4: {args.rows} x 1024 bf16 centroids ({max(64, args.rows // 16)} clusters, sigma 0.07 as whole-"
            f"perturbation length), batch {args.queries} (Zipf 1.0, 20% out-of-distribution), top-4, theta in [0.78, 0.93]")


# ------------------------------------------------------------------------------ multi-rank helpers
def max_over_ranks(value: float, world: int, device=None) -> float:
    """The slowest rank's time: what a whole-job throughput has to be divided by."""
    if world == 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(queries_per_rank: int, world: int, ms_per_step: float) -> float:
    """Queries per second over all ranks (weak scaling: every rank looks up its own batch)."""
    return world * queries_per_rank / (ms_per_step * 1e-3)


# ------------------------------------------------------------------------------ CPU oracle legs
def time_oracle(w, n_sample: int, repeats: int = 1):
    """Seconds per call of the oracle on the first n_sample queries of the batch (all host cores)."""
    import oracle
    q, th = w.queries[:n_sample], w.theta[:n_sample]
    times = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        oracle.lookup(w.centroids, q, th, w.k)
        times.append(time.perf_counter() - t0)
    return times


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    cores = os.cpu_count() or 1
    w = workload(args, 0, cores)
    import oracle
    oracle.build()
    n_sample = max(1, min(args.queries, cores))
    for _ in range(args.warmup):
        time_oracle(w, n_sample)
    t = time_oracle(w, n_sample, args.steps)
    total = sum(t)
    value = n_sample * args.steps / total
    sample = f"{n_sample} of {args.queries} queries per step against all {args.rows} centroids"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_name(args), "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)
    return 0


# ------------------------------------------------------------------------------ clocks
class ClockSampler:
    """nvidia-smi sampled every 50 ms between start and stop(): SM clock (plain median, min and max of ALL samples of
    the window), power and the throttle reasons that were active in any sample."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.proc.stdout.readline()          # the first sample: the sampler is running before the timed region starts
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in out.splitlines():
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
                pw.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no sample inside the timed region"], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_mhz_min": min(sm), "sm_mhz_max": max(sm), "sm_max_mhz": max(mx),
                "power_w_max": max(pw), "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------ DRAM traffic from the committed profile
TRAFFIC_PROFILE = os.path.join(ROOT, "profiles", "lookup_tensor_config4_launches.txt")


def kernel_sources_sha(paths) -> str:
    import hashlib
    h = hashlib.sha256()
    for rel in paths:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def committed_traffic():
    """DRAM bytes per launch of the sweep kernel from the committed ncu capture, or None when the kernel's sources
    have changed since that capture (the profile records their hash): a stale counter is not reported."""
    try:
        fields = {}
        with open(TRAFFIC_PROFILE) as f:
            for ln in f:
                if ln.startswith(("traffic_bytes_per_launch:", "kernel_sources:", "kernel_sources_sha256:")):
                    key, val = ln.split(":", 1)
                    fields[key] = val.strip()
        if kernel_sources_sha(fields["kernel_sources"].split()) != fields["kernel_sources_sha256"]:
            return None
        return float(fields["traffic_bytes_per_launch"])
    except (OSError, KeyError, ValueError):
        return None


# ------------------------------------------------------------------------------ GPU arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2508_18736_b200 import build as _b

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} needs WORLD_SIZE={args.gpus} (launch with torch.distributed.run); got {world}")
    if not torch.cuda.is_available():
        raise SystemExit("no CUDA device: this benchmark has no CPU path (use --impl reference for the oracle)")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if local_rank == 0:
        _b.build()
    if world > 1:
        dist.barrier()
    import paper_2508_18736_b200 as siso

    cores = os.cpu_count() or 1
    w = workload(args, rank, max(1, cores // world))
    B, k = args.queries, w.k
    dev = torch.device("cuda", local_rank)

    def to_dev(a):
        return torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)

    cache = siso.SisoCache(args.rows, 1024, "bf16", device=local_rank)
    step_rows = 1 << 16
    for lo in range(0, args.rows, step_rows):          # promote the centroids in slices: bounded staging
        cache.insert(to_dev(w.centroids[lo:lo + step_rows]))
    cache.check_status()
    cache.set_lookup_path({"auto": siso.PATH_AUTO, "simt": siso.PATH_SIMT, "tensor": siso.PATH_TENSOR,
                           "stream": siso.PATH_STREAM}[args.path])
    q_dev = to_dev(w.queries)
    th_dev = torch.from_numpy(w.theta).to(dev)
    out = (torch.empty((B, k), dtype=torch.int32, device=dev), torch.empty((B, k), dtype=torch.float32, device=dev),
           torch.empty(B, dtype=torch.uint8, device=dev))
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def step_device():
        cache.lookup(q_dev, th_dev, k, out=out)

    # pinned host buffers of the end-to-end leg
    h_q = torch.from_numpy(w.queries.view(np.int16)).pin_memory()
    h_th = torch.from_numpy(w.theta).pin_memory()
    h_idx = torch.empty((B, k), dtype=torch.int32).pin_memory()
    h_sim = torch.empty((B, k), dtype=torch.float32).pin_memory()
    h_hit = torch.empty(B, dtype=torch.uint8).pin_memory()

    def step_host():
        cache.lookup_host(h_q, h_th, 0.0, k, h_idx, h_sim, h_hit)

    def timed(step, steps):
        """Returns (ms per step, per-step ms list, launches) with CUDA events on the launching stream."""
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        barrier()
        l0 = cache.launch_count
        ev[0].record(stream)
        for i in range(steps):
            step()
            ev[i + 1].record(stream)
        barrier()
        per = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
        total = max_over_ranks(ev[0].elapsed_time(ev[steps]), world, dev)
        return total / steps, per, cache.launch_count - l0

    for _ in range(max(3, args.warmup)):
        step_device()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank) if rank == 0 else None        # started after the warm-up
    ms, per_step, launches = timed(step_device, args.steps)
    clocks = sampler.stop() if sampler else None
    cache.check_status()
    legs = {"device": {"ms_per_step": ms, "clocks": clocks}}

    e2e = None
    if not args.no_e2e:
        for _ in range(3):
            step_host()
        torch.cuda.synchronize()
        sampler = ClockSampler(local_rank) if rank == 0 else None
        ms_e2e, _, _ = timed(step_host, args.steps)
        legs["e2e"] = {"ms_per_step": ms_e2e, "clocks": sampler.stop() if sampler else None}
        cache.check_status()
        e2e = {"value": whole_job_value(B, world, ms_e2e), "unit": UNIT,
               "h2d_bytes_per_step": int(w.queries.nbytes + w.theta.nbytes),
               "d2h_bytes_per_step": int(h_idx.numel() * 4 + h_sim.numel() * 4 + h_hit.numel()),
               "ms_per_step": ms_e2e}
        # the host-buffer call must return what the device call returns
        assert torch.equal(h_idx, out[0].cpu()) and torch.equal(h_hit, out[2].cpu())
        # where the end-to-end step's time goes: the same three stages issued one by one with an event after each
        # (host -> device copies of queries and thresholds, the lookup, device -> host copies of the three results)
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
        q_stage, th_stage = torch.empty_like(q_dev), torch.empty_like(th_dev)
        barrier()
        for e in ev:
            e[0].record(stream)
            q_stage.view(torch.int16).copy_(h_q, non_blocking=True)
            th_stage.copy_(h_th, non_blocking=True)
            e[1].record(stream)
            cache.lookup(q_stage, th_stage, k, out=out)
            e[2].record(stream)
            h_idx.copy_(out[0], non_blocking=True)
            h_sim.copy_(out[1], non_blocking=True)
            h_hit.copy_(out[2], non_blocking=True)
            e[3].record(stream)
        barrier()
        e2e["stages_ms"] = {name: statistics.median(e[a].elapsed_time(e[a + 1]) for e in ev)
                            for a, name in enumerate(("h2d_copy", "lookup", "d2h_copy"))}

    # the same device-resident step back to back for at least two seconds: the clock the power cap settles at, and the
    # step time x clock product that makes runs at different clocks comparable
    sustained = None
    if rank == 0 and world == 1:
        n_sus = max(args.steps, int(2200.0 / ms) + 1)
        sampler = ClockSampler(local_rank)
        ms_sus, per_sus, _ = timed(step_device, n_sus)
        ck = sampler.stop()
        sustained = {"steps": n_sus, "ms_per_step": ms_sus, "median_step_ms": statistics.median(per_sus), "clocks": ck,
                     "ms_x_mhz": ms_sus * ck["sm_mhz"] if ck.get("sm_mhz") else None}
        cache.check_status()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    peaks, peak_kind = load_peaks()
    flops = 2.0 * B * args.rows * 1024
    kernel_ms = statistics.median(per_step)           # the sweep kernel plus its small finalize kernel
    achieved = flops / (kernel_ms * 1e-3) / 1e12
    # DRAM bytes per launch of the dominant kernel come from the committed one-pass ncu capture of this very command;
    # they are only known for the full-size workload on the tensor-core kernel, and only while the kernel's sources
    # are the ones that were profiled
    traffic = None
    if args.path in ("auto", "tensor") and args.rows == (1 << 20) and B == 8192:
        traffic = committed_traffic()
    roofline = {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": achieved / peaks["bf16_tflops"], "traffic": traffic,
                "traffic_source": "committed ncu capture (profiles/), not this run" if traffic else None,
                "peak_kind": f"{peak_kind}, burst",
                "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"],
                "hbm_floor_ms": (args.rows * 1024 * 2 + B * 1024 * 2) / (peaks["hbm_gbs"] * 1e9) * 1e3,
                "kernel": {"auto": "tensor-core sweep (auto)", "tensor": "tensor-core sweep", "simt": "CUDA-core sweep",
                           "stream": "streaming sweep"}[args.path],
                "flops_per_launch": flops, "median_launch_ms": kernel_ms}
    if sustained:
        sustained["frac_of_sustained_peak"] = flops / (sustained["ms_per_step"] * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"]
    line = {"metric": METRIC, "value": whole_job_value(B, world, ms), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload_name(args), "parallelism": f"replica x{world}, queries sharded",
                       "l2": "inputs larger than L2: the 2 GiB centroid matrix is swept on every step",
                       "lookup_path": args.path},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "legs": legs,
            "sustained": sustained}

    if world == 1 and not args.no_secondary:
        line["secondary"] = secondary_measurements(args, siso, cache, w, peaks, cores, dev)

    if not args.no_cpu_baseline and world == 1:
        import oracle
        oracle.build()
        n_sample = max(1, min(B, 8 * cores))
        t0 = time.perf_counter()
        o_idx, o_sim, o_hit = oracle.lookup(w.centroids, w.queries[:n_sample], w.theta[:n_sample], k)
        t = time.perf_counter() - t0
        sample = f"first {n_sample} of {B} queries against all {args.rows} centroids, top-{k}"
        line["cpu_baseline"] = {"value": n_sample / t, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                                "seconds": t}
        # the sampled rows double as a full-size parity check of the timed configuration: decisions that differ from
        # the oracle's outside the stated band (2e-3 for bf16), inside it, and outside a band of 1e-5
        g_idx, g_hit = out[0][:n_sample].cpu().numpy(), out[2][:n_sample].cpu().numpy()
        g_sim = out[1][:n_sample].cpu().numpy().astype(np.float64)
        diff = g_idx != o_idx
        short = np.where(diff, np.abs(o_sim - g_sim), 0.0)       # how far the differing slot falls short of the rank's best
        margin = np.abs(o_sim[:, 0] - w.theta[:n_sample].astype(np.float64))
        hit_diff = g_hit != o_hit
        line["parity_sample"] = {"rows": n_sample, "max_sim_err": float(np.abs(g_sim - o_sim).max()),
                                 "top1_equal": int((g_idx[:, 0] == o_idx[:, 0]).sum()), "hit_equal": int((~hit_diff).sum()),
                                 "outside_band": int((short > 2e-3).sum() + (hit_diff & (margin >= 2e-3)).sum()),
                                 "excused": int(diff.sum() + hit_diff.sum()),
                                 "strict_mismatch": int((short > 1e-5).sum() + (hit_diff & (margin >= 1e-5)).sum())}
    print(json.dumps(line), flush=True)
    cache.close()
    if world > 1:
        dist.destroy_process_group()
    return 0


# ------------------------------------------------------------------------------ the rest of the target, in the default line
def _time_ms(torch, fn, steps, warm):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def small_batch_sweep(torch, cache, queries_dev, rows, dim, peaks, batches=(1, 8, 128, 256), steps=20, warm=3):
    """Top-1 lookups of a few queries: the centroid matrix is streamed from HBM once per call."""
    out = []
    for b in batches:
        q = queries_dev[:b].contiguous()
        ms = _time_ms(torch, lambda: cache.lookup(q, 0.86, 1), steps, warm)
        gbs = rows * dim * 2 / ms / 1e6
        rec = {"batch": b, "us": round(ms * 1e3, 2), "GB/s": round(gbs, 1), "frac": round(gbs / peaks["hbm_gbs"], 4)}
        if b >= 256:
            # at 256 queries the sweep sits on the ridge (flop per centroid byte = 256): say where it stands against the
            # tensor roof too; the binding roof is the larger of the two times
            tf = 2.0 * b * rows * dim / ms / 1e9
            rec["TFLOP/s"] = round(tf, 1)
            rec["frac_tensor"] = round(tf / peaks["bf16_tflops"], 4)
        out.append(rec)
    return out


def config5_steady_state(torch, siso, W, peaks, cores, dev, n_warm=400, n_timed=1200):
    """The streaming step on a full cache (262,144 x 768 bf16, micro-batches of 256): lookup, hit update, eviction of
    what the misses lack, insertion of the misses.  Returns (result dict, cache, one batch of queries on the device)."""
    sp = W.StreamSpec()
    stream = W.QueryStream(sp, threads=cores)

    def to_dev(a):
        return torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)

    q_all = to_dev(stream.block(0, n_warm + n_timed, threads=cores))
    cache = siso.SisoCache(sp.capacity, sp.dim, "bf16")
    # the stream starts on an empty cache; to time the steady state (full cache, evicting every batch) the cache is
    # first filled with later queries of the same stream
    filler = stream.block(20000, 20000 + (sp.capacity - 2048) // sp.batch, threads=cores)
    for lo in range(0, filler.shape[0], 1 << 16):
        cache.insert(to_dev(filler[lo:lo + (1 << 16)]))
    cache.check_status()
    out = None
    for t in range(n_warm):
        out = cache.stream_step(q_all[t * 256:(t + 1) * 256], float(sp.theta), out=out)
    torch.cuda.synchronize()
    s0, l0 = cache.stats(), cache.launch_count
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for t in range(n_warm, n_warm + n_timed):
        out = cache.stream_step(q_all[t * 256:(t + 1) * 256], float(sp.theta), out=out)
    e1.record()
    torch.cuda.synchronize()
    cache.check_status()
    s1 = cache.stats()
    us = e0.elapsed_time(e1) / n_timed * 1e3
    gbs = sp.capacity * sp.dim * 2 / (us * 1e-6) / 1e9
    res = {"workload": "config 5 steady state: 262,144 x 768 bf16 cache, full; micro-batches of 256 (lookup, hit update, "
                       "eviction, insertion of the misses)",
           "us_per_batch": us, "queries_per_s": 256 / us * 1e6, "batches_timed": n_timed,
           "hit_ratio": (s1["hits"] - s0["hits"]) / (256.0 * n_timed), "evictions": s1["evictions"] - s0["evictions"],
           "inserts": s1["inserts"] - s0["inserts"], "launches_per_batch": (cache.launch_count - l0) / n_timed,
           "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": gbs / peaks["hbm_gbs"],
                        "note": "384 MiB of centroids per micro-batch over the whole step time; at 256 queries the step "
                                "also sits on the tensor roof (flop per centroid byte = 256 against a ridge near 250)"}}
    return res, cache, q_all[:256]


def secondary_measurements(args, siso, cache4, w4, peaks, cores, dev):
    """What the target names besides the headline: the streaming paths against the HBM roof (small-batch sweeps of both
    stated matrices, the whole streaming step of configuration 5) and the hit update of configuration 2."""
    import torch
    from gen import workloads as W
    t_start = time.perf_counter()
    sec = {}

    def to_dev(a):
        return torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)

    cache4.set_lookup_path(siso.PATH_AUTO)
    sec["small_batch_1048576x1024"] = small_batch_sweep(torch, cache4, to_dev(w4.queries[:256]), args.rows, 1024, peaks)
    c5, cache5, q5 = config5_steady_state(torch, siso, W, peaks, cores, dev)
    sec["config5"] = c5
    sec["small_batch_262144x768"] = small_batch_sweep(torch, cache5, q5, 262144, 768, peaks)
    cache5.close()
    # configuration 2: lookup, then the running-mean update of the hit centroids (65,536 queries into 65,536 rows)
    w2 = W.config(2, threads=cores)
    cache2 = siso.SisoCache(65536, 768, "bf16")
    cache2.insert(to_dev(w2.centroids))
    q, th = to_dev(w2.queries), torch.from_numpy(w2.theta).to(dev)
    ms_l = _time_ms(torch, lambda: cache2.lookup(q, th, 1), 10, 3)
    idx, sim, hit = cache2.lookup(q, th, 1)
    times = []
    for _ in range(7):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        cache2.update(q, idx, hit)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    cache2.check_status()
    n_hit = int(hit.sum().item())
    touched = int(torch.unique(idx[hit.bool(), 0]).numel())
    upd_bytes = n_hit * 768 * 2 + touched * 768 * (4 + 4 + 2)        # hit queries read; master read + written, copy written
    ms_u = statistics.median(times[2:])
    sec["config2"] = {"workload": "config 2: 65,536 x 768 bf16, batch 65,536, Zipf 1.1, theta in [0.80, 0.92]",
                      "lookup_ms": ms_l, "update_ms": ms_u, "hits": n_hit, "centroids_touched": touched,
                      "lookup_frac_of_bf16_peak": 2.0 * 65536 * 65536 * 768 / ms_l / 1e9 / peaks["bf16_tflops"],
                      "update_roofline": {"bound": "hbm", "achieved": upd_bytes / ms_u / 1e6, "peak": peaks["hbm_gbs"],
                                          "unit": "GB/s", "frac": upd_bytes / ms_u / 1e6 / peaks["hbm_gbs"]}}
    cache2.close()
    sec["seconds"] = time.perf_counter() - t_start
    return sec


# ------------------------------------------------------------------------------ the centroid-sharded cache
def run_sharded(args):
    """One JSON line for the cache partitioned over the ranks (sharded.py): config-4 lookup with the rows split N ways
    and the sharded streaming step of configuration 5.  Launched like the default arm (torchrun for N > 1)."""
    import torch
    import torch.distributed as dist
    from paper_2508_18736_b200 import build as _b
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} needs WORLD_SIZE={args.gpus} (launch with torch.distributed.run); got {world}")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if local_rank == 0:
        _b.build()
    if world > 1:
        dist.barrier()
    import paper_2508_18736_b200 as siso
    from gen import workloads as W
    cores = max(1, (os.cpu_count() or 1) // world)
    peaks, peak_kind = load_peaks()

    def to_dev(a):
        return torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(step, steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for _ in range(steps):
            step()
        e1.record()
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), world, dev) / steps

    # ---- lookup: the same centroids and the same batch on every rank (seeded), each rank keeps its rows
    w = workload(args, 0, cores)
    B, k = args.queries, w.k
    shard = siso.ShardedCache(args.rows, 1024, "bf16", device=local_rank)
    for lo in range(shard.lo, shard.hi, 1 << 16):
        hi = min(shard.hi, lo + (1 << 16))
        shard.local.insert(to_dev(w.centroids[lo:hi]))
    shard.local.check_status()
    q, th = to_dev(w.queries), torch.from_numpy(w.theta).to(dev)
    for _ in range(max(3, args.warmup)):
        shard.lookup(q, th, k)
    sampler = ClockSampler(local_rank) if rank == 0 else None
    ms = timed(lambda: shard.lookup(q, th, k), args.steps)
    clocks = sampler.stop() if sampler else None
    idx, sim, hit = shard.lookup(q, th, k)
    shard.local.check_status()
    flops = 2.0 * B * args.rows * 1024
    line = {"metric": METRIC + " (centroid-sharded cache)", "value": B / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True, "scaling": "strong",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload_name(args), "parallelism": f"centroid rows sharded x{world}: {shard.hi - shard.lo} rows per rank, "
                       "every rank scores the whole batch, one all-gather of packed top-k keys",
                       "l2": "inputs larger than L2 while rows / ranks x 2 KiB exceeds it"},
            "clocks": clocks, "hits": int(hit.sum().item()),
            "roofline": {"bound": "tensor", "achieved": flops / (ms * 1e-3) / 1e12, "peak": peaks["bf16_tflops"] * world, "unit": "TFLOP/s",
                         "frac": flops / (ms * 1e-3) / 1e12 / (peaks["bf16_tflops"] * world), "traffic": None,
                         "peak_kind": f"{peak_kind}, burst, x{world} GPUs"}}
    shard.close()
    # ---- the sharded streaming step (configuration 5's cache split over the ranks, steady state)
    sp = W.StreamSpec()
    stream = W.QueryStream(sp, threads=cores)
    n_warm, n_timed = 100, 300
    q_all = to_dev(stream.block(0, n_warm + n_timed, threads=cores))
    sc = siso.ShardedCache(sp.capacity, sp.dim, "bf16", device=local_rank)
    first = 20000 + sc.lo // sp.batch
    filler = stream.block(first, first + (sc.hi - sc.lo) // sp.batch, threads=cores)
    for lo in range(0, filler.shape[0], 1 << 16):
        sc.local.insert(to_dev(filler[lo:lo + (1 << 16)]))
    sc.local.check_status()
    t = [0]

    def stream_step():
        sc.stream_step(q_all[t[0] * 256:(t[0] + 1) * 256], float(sp.theta))
        t[0] += 1

    for _ in range(n_warm):
        stream_step()
    us = timed(stream_step, n_timed) * 1e3
    st = sc.local.stats()
    line["stream_step"] = {"workload": f"config 5 cache ({sp.capacity} x {sp.dim} bf16) sharded x{world}, micro-batches of 256",
                           "us_per_batch": us, "queries_per_s": 256 / us * 1e6, "evictions_this_rank": st["evictions"],
                           "note": "lookup keys, free counts, eviction keys and slots are exchanged every batch; the miss count, "
                                   "the free slots and the number of entries to evict stay on the device (no host read in the step)"}
    sc.close()
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
    return 0


# ------------------------------------------------------------------------------ the other configurations
def run_other(args):
    """One JSON line for configuration 1, 2, 3, 5 or the small-batch streaming probe (single GPU, device-resident)."""
    import torch
    from paper_2508_18736_b200 import build as _b
    _b.build()
    import paper_2508_18736_b200 as siso
    from gen import workloads as W
    peaks, peak_kind = load_peaks()
    cores = os.cpu_count() or 1
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)

    def to_dev(a, dtype):
        if dtype == "bf16":
            return torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)
        return torch.from_numpy(a).to(dev)

    def fill(cache, cent, dtype):
        for lo in range(0, cent.shape[0], 1 << 16):
            cache.insert(to_dev(cent[lo:lo + (1 << 16)], dtype))
        cache.check_status()

    def time_ms(fn, steps, warm):
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps

    steps, warm = args.steps, max(3, args.warmup)
    line = {"workload": args.workload, "n_gpus": 1, "steps": steps, "warmup": warm, "data": "synthetic",
            "peaks": peak_kind}
    props = torch.cuda.get_device_properties(0)
    # nominal: SMs x 128 FP32 lanes x 2 flop x max SM clock; measured: the library's register-only FMA kernel
    fp32_nominal = props.multi_processor_count * 128 * 2 * (getattr(props, "clock_rate", 1965000) * 1e3) / 1e12
    probe = siso.SisoCache(64, 64, "f32")
    fp32_peak = {"measured_tflops": probe.measure_fp32_fma(), "nominal_tflops": fp32_nominal,
                 "sm_count": props.multi_processor_count}
    probe.close()

    def oracle_baseline(fn, value_of, unit, sample):
        """The CPU oracle as it stands, timed once on the host cores beside the GPU number."""
        if args.no_cpu_baseline:
            return None
        import oracle
        oracle.build()
        t0 = time.perf_counter()
        res = fn(oracle)
        t = time.perf_counter() - t0
        return {"value": value_of(t), "unit": unit, "cores": cores, "kind": "oracle", "sample": sample, "seconds": t}, res
    if args.workload == "config1":
        w = W.config(1)
        cache = siso.SisoCache(1024, 384, "f32")
        fill(cache, w.centroids, "f32")
        q = to_dev(w.queries, "f32")
        ms = time_ms(lambda: cache.lookup(q, 0.85, 1), steps, warm)
        fl = 2.0 * 4096 * 1024 * 384
        tc_peak = peaks["bf16_tflops"] / 3.0     # fp32 products as three bf16 MMAs (split-bf16 selection + exact rescoring)
        line.update(metric="lookup queries/s, 1,024 x 384 fp32, batch 4,096", value=4096 / ms * 1e3, unit=UNIT,
                    ms_per_step=ms, dtype="f32", rescans=cache.stats()["rescans"],
                    roofline={"bound": "tensor", "achieved": fl / ms / 1e9, "peak": tc_peak, "unit": "TFLOP/s",
                              "frac": fl / ms / 1e9 / tc_peak, "traffic": None,
                              "peak_kind": "measured bf16 burst peak / 3 (split-bf16 emulation of fp32 products)",
                              "note": "3.2 GFLOP in six launches: a launch-latency-sized problem (one tile per CTA)",
                              "fp32_alu_peak": fp32_peak})
        cb = oracle_baseline(lambda o: o.lookup(w.centroids, w.queries, w.theta, 1), lambda t: 4096 / t, UNIT,
                             "the whole batch: 4,096 queries against 1,024 centroids")
        if cb:
            line["cpu_baseline"] = cb[0]
    elif args.workload == "config2":
        w = W.config(2, threads=cores)
        cache = siso.SisoCache(65536, 768, "bf16")
        fill(cache, w.centroids, "bf16")
        q, th = to_dev(w.queries, "bf16"), torch.from_numpy(w.theta).to(dev)
        ms_l = time_ms(lambda: cache.lookup(q, th, 1), steps, warm)
        idx, sim, hit = cache.lookup(q, th, 1)
        ms_u = time_ms(lambda: cache.update(q, idx, hit), max(3, steps // 4), 1)
        fl = 2.0 * 65536 * 65536 * 768
        line.update(metric="lookup + update queries/s, 65,536 x 768 bf16, batch 65,536", value=65536 / (ms_l + ms_u) * 1e3,
                    unit=UNIT, ms_per_step=ms_l + ms_u, lookup_ms=ms_l, update_ms=ms_u, dtype="bf16",
                    hit_ratio=float(hit.float().mean().item()),
                    roofline={"bound": "tensor", "achieved": fl / ms_l / 1e9, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                              "frac": fl / ms_l / 1e9 / peaks["bf16_tflops"], "kernel": "lookup only"})
        n_s = min(65536, 64 * cores)
        cb = oracle_baseline(lambda o: o.lookup(w.centroids, w.queries[:n_s], w.theta[:n_s], 1), lambda t: n_s / t, UNIT,
                             f"lookup of the first {n_s} of 65,536 queries against all 65,536 centroids")
        if cb:
            line["cpu_baseline"] = cb[0]
            import oracle
            oc = oracle.OracleCache(65536, 768, "bf16")
            oc.insert(w.centroids)
            i_np, h_np = idx.cpu().numpy(), hit.cpu().numpy()
            t0 = time.perf_counter()
            oc.update(w.queries, i_np, h_np)
            line["cpu_baseline"]["update_seconds"] = time.perf_counter() - t0
            line["cpu_baseline"]["update_sample"] = "the whole batch of 65,536 queries with the GPU's decisions"
    elif args.workload == "config3":
        w = W.config(3, threads=cores)
        cache = siso.SisoCache(32768, 768, "f32")
        fill(cache, w.centroids, "f32")
        st = cache.export()
        times, merged = [], None
        for _ in range(max(3, steps // 4)):
            cache.import_(st["master"], st["size"], st["access"], st["last"], st["valid"], 0)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            _, merged = cache.merge(W.MERGE_THRESHOLD_CONFIG3, siso.MERGE_WEIGHTED_MEAN)
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        ms = statistics.median(times)
        fl = 32768.0 * 32767 / 2 * 768 * 2
        # the sweep is a bf16 filter on the tensor cores (one product per pair of rows and K step, rows rounded to bf16, margin
        # = the bound of that rounding) and the exact fp32 check decides: the tensor work is one bf16 multiply-add per
        # algorithmic one, so the peak is the measured bf16 peak itself
        tc_peak = peaks["bf16_tflops"]
        line.update(metric="self-merge pass, 32,768 x 768 fp32, theta_C 0.90, weighted mean", value=32768 / ms * 1e3,
                    unit="centroids/s", ms_per_step=ms, merged=merged, survivors=cache.stats()["occupancy"], dtype="f32",
                    roofline={"bound": "tensor", "achieved": fl / ms / 1e9, "peak": tc_peak, "unit": "TFLOP/s",
                              "frac": fl / ms / 1e9 / tc_peak, "traffic": None,
                              "peak_kind": "measured bf16 burst peak (one bf16 product per pair; the exact check touches candidates only)",
                              "note": "whole pass (rounding, sweep, exact check, grouping, resolution, apply) over the "
                                      "lower-triangle flops N(N-1)/2 x 2D; the sweep kernel is about two thirds of it",
                              "fp32_alu_peak": fp32_peak})

        def whole_merge(o):
            oc = o.OracleCache(32768, 768, "f32")
            oc.insert(w.centroids)
            return oc.merge(W.MERGE_THRESHOLD_CONFIG3, True)

        cb = oracle_baseline(whole_merge, lambda t: 32768 / t, "centroids/s", "the whole pass over all 32,768 centroids")
        if cb:
            line["cpu_baseline"] = cb[0]
            line["cpu_baseline"]["merged_equal"] = bool(cb[1][1] == merged)
    elif args.workload == "f32_lookup":
        # an fp32 cache at scale: 262,144 x 1024 fp32 centroids (1 GiB), batch 4,096, top-4; clusters as in configuration 4
        N = 262144 if args.rows == (1 << 20) else args.rows
        B = 4096 if args.queries == 8192 else args.queries
        D = 1024
        w = W.config(1, threads=cores, n_centroids=N, n_queries=B, dim=D, n_clusters=max(2, N // 16), theta=(0.78, 0.93), k=4)
        cache = siso.SisoCache(N, D, "f32")
        fill(cache, w.centroids, "f32")
        q, th = to_dev(w.queries, "f32"), torch.from_numpy(w.theta).to(dev)
        res = {}
        for name, path in (("cuda_cores", siso.PATH_SIMT), ("tensor", siso.PATH_TENSOR)):
            cache.set_lookup_path(path)
            res[name] = time_ms(lambda: cache.lookup(q, th, 4), steps if name == "tensor" else max(3, steps // 4), warm)
        ms = res["tensor"]
        fl = 2.0 * N * B * D
        tc_peak = peaks["bf16_tflops"] / 3.0
        line.update(metric=f"lookup queries/s, {N:,} x {D} fp32, batch {B:,}, top-4", value=B / ms * 1e3, unit=UNIT, ms_per_step=ms,
                    cuda_core_sweep_ms=res["cuda_cores"], rescans=cache.stats()["rescans"], dtype="f32",
                    roofline={"bound": "tensor", "achieved": fl / ms / 1e9, "peak": tc_peak, "unit": "TFLOP/s",
                              "frac": fl / ms / 1e9 / tc_peak, "traffic": None,
                              "peak_kind": "measured bf16 burst peak / 3 (split-bf16 emulation of fp32 products)",
                              "fp32_alu_peak": fp32_peak})
    elif args.workload == "tiered":
        # locality-ordered exact search (the exact counterpart of the Sec. 4.3 placement): a merged cache of 524,288 x 1024
        # bf16 centroids (one per cluster, 1 GiB), cluster_size grown by 8 batches of hits, hot tier = the 1/16 of the
        # entries FilteringCentroids would evict last; batches of 8,192 queries (Zipf 1.0, 20 % out of distribution)
        N = 524288 if args.rows == (1 << 20) else args.rows
        B, D, warm_batches = args.queries, 1024, 8
        w = W.config(4, threads=cores, n_centroids=16, n_queries=B * (warm_batches + 1), dim=D, n_clusters=N)
        cent = W.f32_to_bf16_bits(W.unit_gaussian_rows(N, D, 0, W._TAG_MEANS, cores))      # the cluster means themselves
        cache = siso.SisoCache(N, D, "bf16")
        fill(cache, cent, "bf16")
        q_all, th_all = to_dev(w.queries, "bf16"), torch.from_numpy(w.theta).to(dev)
        for t in range(warm_batches):
            qb, tb = q_all[t * B:(t + 1) * B], th_all[t * B:(t + 1) * B]
            idx, sim, hit = cache.lookup(qb, tb, 1)
            cache.update(qb, idx, hit)
        # MergeCentroids at 0.5 finds nothing to merge: every pair of entries is at most 0.5 similar (checked in fp64)
        sep = 0.5
        _, merged = cache.merge(sep, siso.MERGE_WEIGHTED_MEAN)
        assert merged == 0, merged
        tiers = siso.TieredCache(cache, N // 16, sep + 4e-3, 2e-3)          # bf16 rounding of the fp32 masters: 4e-3, norms 2e-3
        q, th = q_all[warm_batches * B:], th_all[warm_batches * B:]
        ms_full = time_ms(lambda: cache.lookup(q, th, 1), steps, warm)
        ms = time_ms(lambda: tiers.lookup(q, th), steps, warm)
        a, b = cache.lookup(q, th, 1), tiers.lookup(q, th)
        same = bool((a[0][:, 0] == b[0]).all().item() and (a[2] == b[2]).all().item())
        n_go = B - tiers.settled
        fl = 2.0 * D * (B * tiers.n_hot + n_go * tiers.n_cold)
        line.update(metric=f"lookup queries/s, locality-ordered exact search, {N:,} x {D} bf16, hot tier {tiers.n_hot:,}, batch {B:,}, top-1",
                    value=B / ms * 1e3, unit=UNIT, ms_per_step=ms, whole_cache_ms=ms_full, speedup=ms_full / ms,
                    ended_in_hot_tier=tiers.settled / B, exit_similarity=tiers.exit_sim, equal_to_whole_cache_lookup=same, dtype="bf16",
                    roofline={"bound": "tensor", "achieved": fl / ms / 1e9, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                              "frac": fl / ms / 1e9 / peaks["bf16_tflops"], "traffic": None,
                              "note": "products actually computed (all queries x hot tier + remaining queries x cold tier)"})
    elif args.workload == "evict":
        # FilteringCentroids on the configuration-5 cache: the 256 lowest (cluster_size, access_count, last_access, slot)
        # keys of 262,144 entries, then the decay pass; entries are put back between calls
        sp = W.StreamSpec()
        n, dim, m = sp.capacity, sp.dim, 256
        cache = siso.SisoCache(n, dim, "bf16")
        rows = torch.randn(1 << 16, dim, device=dev).to(torch.bfloat16)
        sizes = torch.from_numpy(np.random.default_rng(0).integers(1, 64, n).astype(np.float64)).to(dev)
        for lo in range(0, n, 1 << 16):
            cache.insert(rows, sizes[lo:lo + (1 << 16)])
        refill = rows[:m].contiguous()
        times_e, times_d = [], []
        for it in range(steps + warm):
            e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            e0.record()
            cache.evict(m)
            e1.record()
            cache.evict(0, siso.EVICT_DECAY)
            e2.record()
            torch.cuda.synchronize()
            cache.insert(refill)
            if it >= warm:
                times_e.append(e0.elapsed_time(e1)); times_d.append(e1.elapsed_time(e2))
        ms_e, ms_d = statistics.median(times_e), statistics.median(times_d)
        meta = n * 21.0                                  # cluster_size 8 + access_count 4 + last_access 8 + live flag 1
        line.update(metric=f"eviction of the {m} lowest keys of {n:,} entries (exact selection); decay pass", value=n / ms_e * 1e3,
                    unit="entries/s", ms_per_step=ms_e, decay_ms=ms_d, dtype="u64 keys / f64 sizes",
                    roofline={"bound": "hbm", "achieved": 2 * meta / ms_e / 1e6, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                              "frac": 2 * meta / ms_e / 1e6 / peaks["hbm_gbs"], "traffic": None,
                              "note": "two scans of 21 bytes of metadata per entry (5.5 MB each): a launch-latency-sized problem"})
    elif args.workload == "cluster":
        # stand-in for the query log that SISO-Cluster turns into centroids (Sec. 4.1): 131,072 unit vectors of dim 768
        # around 13,107 cluster means (the paper's 10 queries per centroid), clustered at theta_C = 0.86
        n, dim = (131072 if args.rows == (1 << 20) else args.rows), 768
        w = W.config(3, threads=cores, n_centroids=n, dim=dim, n_clusters=max(2, n // 10), sigma=0.06, dtype=args.dtype)
        cache = siso.SisoCache(64, dim, args.dtype)
        v = to_dev(w.centroids, args.dtype)
        times, k = [], 0
        for it in range(max(3, steps // 4) + 1):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            label, centres, sizes, cent = cache.cluster(v, 0.86)
            e1.record()
            torch.cuda.synchronize()
            if it > 0:
                times.append(e0.elapsed_time(e1))
            k = len(centres)
        ms = statistics.median(times)
        fl = float(n) * (n - 1) / 2 * dim * 2
        tc_peak = peaks["bf16_tflops"]       # fp32 rows too: the sweep is a one-product bf16 filter, the exact check decides
        planted = int(len(np.unique(w.centroid_labels)))
        line.update(metric=f"community detection, {n:,} x {dim} {args.dtype} vectors, theta_C 0.86 (all pairs, order, founders, mean centroids)",
                    value=n / ms * 1e3, unit="vectors/s", ms_per_step=ms, communities=k, planted_clusters=planted, dtype=args.dtype,
                    roofline={"bound": "tensor", "achieved": fl / ms / 1e9, "peak": tc_peak, "unit": "TFLOP/s",
                              "frac": fl / ms / 1e9 / tc_peak, "traffic": None,
                              "peak_kind": "measured bf16 burst peak (whole call: sweep, exact check, order, founders, means)"})
    elif args.workload == "config5_full":
        # the whole stream of configuration 5 from an empty cache: 10,000,000 queries in micro-batches of 256, popularity
        # reshuffled every 1,000,000 queries.  Queries are generated a million at a time on the host (not timed), copied
        # to the device, and the steps of that chunk are timed with CUDA events.
        sp = W.StreamSpec(seed=args.seed)
        stream = W.QueryStream(sp, threads=cores)
        cache = siso.SisoCache(sp.capacity, sp.dim, "bf16")
        per_chunk = 3906                                      # batches per chunk (about one popularity epoch)
        total_ms, done, out = 0.0, 0, None
        epochs, first_full, prev, maintenance = [], None, cache.stats(), []
        while done < sp.n_batches:
            stop = min(sp.n_batches, done + per_chunk)
            q = to_dev(stream.block(done, stop, threads=cores), "bf16")
            th_all = None
            if args.theta_range is not None:                   # theta_b ~ U[lo, hi], seeded per chunk
                th_all = torch.from_numpy(W.thresholds(q.shape[0], args.theta_range[0], args.theta_range[1],
                                                       1000 * args.seed + len(epochs))).to(dev)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for t in range(done, stop):
                lo = (t - done) * sp.batch
                qb = q[lo:lo + sp.batch]
                if qb.shape[0] != sp.batch:
                    out = None                                 # the last batch is short
                out = cache.stream_step(qb, float(sp.theta) if th_all is None else th_all[lo:lo + qb.shape[0]], out=out)
            e1.record()
            torch.cuda.synchronize()
            total_ms += e0.elapsed_time(e1)
            st = cache.stats()
            nq = st["lookups"] - prev["lookups"]
            epochs.append({"queries": nq, "hit_ratio": round((st["hits"] - prev["hits"]) / max(1, nq), 4),
                           "inserts": st["inserts"] - prev["inserts"], "evictions": st["evictions"] - prev["evictions"],
                           "us_per_batch": round(e0.elapsed_time(e1) / (stop - done) * 1e3, 1), "occupancy": st["occupancy"]})
            if first_full is None and st["occupancy"] == sp.capacity:
                first_full = len(epochs)
            prev, done = st, stop
            if args.maintain and done < sp.n_batches:
                m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                m0.record()
                _, n_merged = cache.merge(0.86, siso.MERGE_WEIGHTED_MEAN)
                cache.evict(0, siso.EVICT_DECAY)
                m1.record()
                torch.cuda.synchronize()
                cache.check_status()
                maintenance.append({"after_queries": done * sp.batch, "merged": n_merged, "ms": round(m0.elapsed_time(m1), 2),
                                    "occupancy_after": cache.stats()["occupancy"]})
                prev = cache.stats()
        cache.check_status()
        st = cache.stats()
        assert st["lookups"] == sp.n_queries and st["inserts"] - st["evictions"] - st["merges"] == st["occupancy"] <= sp.capacity
        us = total_ms / sp.n_batches * 1e3
        gbs = sp.capacity * sp.dim * 2 / (us * 1e-6) / 1e9
        line.update(metric="streaming cache, whole stream: 10,000,000 queries, 262,144 x 768 bf16, micro-batches of 256, from an empty cache",
                    value=sp.n_queries / total_ms * 1e3, unit=UNIT, us_per_batch=us, batches=sp.n_batches, seed=args.seed, dtype="bf16",
                    theta=float(sp.theta) if args.theta_range is None else f"uniform in [{args.theta_range[0]}, {args.theta_range[1]}] per query",
                    hit_ratio=st["hits"] / sp.n_queries, inserts=st["inserts"], evictions=st["evictions"],
                    cache_full_after_chunk=first_full, chunks=epochs, merges=st["merges"], maintenance=maintenance,
                    maintenance_ms_total=sum(m["ms"] for m in maintenance),
                    roofline={"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                              "frac": gbs / peaks["hbm_gbs"], "traffic": None,
                              "note": "384 MiB of centroid slots per batch over the whole step time (the early batches sweep a partly empty cache)"})
    elif args.workload == "config5":
        sp = W.StreamSpec()
        stream = W.QueryStream(sp, threads=cores)
        n_warm, n_timed = 600, min(4000, max(500, steps * 100))
        q_all = to_dev(stream.block(0, n_warm + n_timed, threads=cores), "bf16")
        cache = siso.SisoCache(sp.capacity, sp.dim, "bf16")
        # the stream starts on an empty cache; to time the steady state (full cache, evicting every batch) the cache
        # is first filled with later queries of the same stream
        fill(cache, stream.block(20000, 20000 + (sp.capacity - 2048) // sp.batch, threads=cores), "bf16")
        out = None
        for t in range(n_warm):
            out = cache.stream_step(q_all[t * 256:(t + 1) * 256], float(sp.theta), out=out)
        torch.cuda.synchronize()
        s0, l0 = cache.stats(), cache.launch_count
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for t in range(n_warm, n_warm + n_timed):
            out = cache.stream_step(q_all[t * 256:(t + 1) * 256], float(sp.theta), out=out)
        e1.record()
        torch.cuda.synchronize()
        cache.check_status()
        s1 = cache.stats()
        us = e0.elapsed_time(e1) / n_timed * 1e3
        gbs = sp.capacity * sp.dim * 2 / (us * 1e-6) / 1e9
        line.update(metric="streaming cache queries/s, 262,144 x 768 bf16, micro-batches of 256 (lookup, update, evict, insert)",
                    value=256 / us * 1e6, unit=UNIT, us_per_batch=us, batches_timed=n_timed, dtype="bf16",
                    hit_ratio=(s1["hits"] - s0["hits"]) / (256.0 * n_timed), evictions=s1["evictions"] - s0["evictions"],
                    inserts=s1["inserts"] - s0["inserts"], gpu_launches=cache.launch_count - l0,
                    roofline={"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                              "frac": gbs / peaks["hbm_gbs"], "traffic": None,
                              "note": "384 MiB of centroids per batch over the whole step time"})
    else:   # stream_probe
        rows = []
        # the two stated matrices; an explicit --rows probes that many rows x 1024 only (small profiler captures)
        for (N, D) in (((1 << 20, 1024), (262144, 768)) if args.rows == (1 << 20) else ((args.rows, 1024),)):
            cache = siso.SisoCache(N, D, "bf16")
            w = W.config(4, threads=cores, n_centroids=N, dim=D, n_queries=256, n_clusters=max(64, N // 16))
            fill(cache, w.centroids, "bf16")
            for B in (1, 2, 4, 8, 16, 32, 64, 128, 256):
                q = to_dev(w.queries[:B], "bf16")
                ms = time_ms(lambda: cache.lookup(q, 0.86, 1), steps, warm)
                gbs = N * D * 2 / ms / 1e6
                rows.append({"rows": N, "dim": D, "batch": B, "us": ms * 1e3, "GB/s": gbs, "frac": gbs / peaks["hbm_gbs"]})
            cache.close()
        line.update(metric="small-batch lookup: centroid bytes per second", unit="GB/s", rows=rows, dtype="bf16",
                    value=max(r["GB/s"] for r in rows),
                    roofline={"bound": "hbm", "peak": peaks["hbm_gbs"], "unit": "GB/s",
                              "achieved": max(r["GB/s"] for r in rows), "frac": max(r["frac"] for r in rows)})
    print(json.dumps(line), flush=True)
    return 0


def main():
    args = parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.sharded:
        return run_sharded(args)
    if args.workload != "config4":
        return run_other(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
