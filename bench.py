#!/usr/bin/env python
"""Benchmark of the SJA advertise / signal / select / commit round.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 0..4] [--impl ours|reference]

One "step" is one pass of the whole round over one synthetic workload: the segmented scan
of all job profiles (sja_load_profiles), sja_advertise, sja_select and sja_commit.
Metric: job-gap pairs evaluated per second (G*J pairs per step; every pair counts, however
early it is declined).  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2509_19086_b200 import replicas  # noqa: E402
from paper_2509_19086_b200 import workloads as wl  # noqa: E402

METRIC = "job-gap pairs evaluated/s"
UNIT = "pairs/s"
POLICY_NAMES = {0: "efficiency", 1: "fairness", 2: "sla"}
# kernels launched per step: count_boundaries, cta_offsets, row_offsets, init_state, scan_profiles | sort_gap_tiles,
# rank_gap_tiles, place_gaps, count_classes | select_tile (or select_merge / select_search), finalize_awards |
# commit_vote, commit_apply, commit_refresh
KERNELS_PER_STEP = 14
FALLBACK_HBM_GBS = 6650.0
# DRAM traffic of the scan kernel from its ncu capture on the 8192-job case (profiles/
# scan_profiles_kernel_cfg2-jobs8192.md): dram__bytes_read.sum + dram__bytes_write.sum over 33 554 432 steps.
# Traffic grows in proportion to the step count, so a full launch is this figure times N.  It is only reported
# while csrc/sja_scan.cuh is the file the counters were taken from (first 16 hex digits of its sha256).
NCU_SCAN_TRAFFIC_BYTES_PER_STEP = (273.045760e6 + 60.581120e6) / 33554432
NCU_SCAN_SOURCE_SHA = "8b4aa85b4bb68d65"


# Issue-slot roofline of the select kernel (it is bound by instruction issue, not HBM): warp instructions of one
# launch on the large uniform workload from ncu (profiles/select_tile_kernel_cfg2-jobs32768.md, full-size line),
# peak = SMs x 4 schedulers x SM clock.  The kernel's work is not proportional to the pair count, so the figure
# holds for that workload only; it is reported while csrc/sja_tile.cuh is the file the counters were taken from
# (its code: the hash was re-taken after a comment-only edit).
NCU_TILE_WARP_INSTR_PER_LAUNCH = 90569842
NCU_TILE_PAIRS = 65536 * 4096
NCU_TILE_SOURCE_SHA = "9470af5ea551c4a3"
N_SM, SCHEDULERS_PER_SM = 148, 4


def _source_sha(name: str):
    import hashlib
    path = os.path.join(ROOT, "paper_2509_19086_b200", "csrc", name)
    try:
        return hashlib.sha256(open(path, "rb").read()).hexdigest()[:16]
    except OSError:
        return None


def select_roofline(pairs, select_ms, sm_mhz):
    """Issue rate of the select kernel against the GPU's warp-instruction issue peak (select_ms also holds the
    few microseconds of finalize_awards_kernel, so the rate is slightly understated)."""
    if not select_ms or pairs != NCU_TILE_PAIRS or _source_sha("sja_tile.cuh") != NCU_TILE_SOURCE_SHA:
        return None
    mhz = sm_mhz or 1965.0
    peak = N_SM * SCHEDULERS_PER_SM * mhz * 1e6
    achieved = NCU_TILE_WARP_INSTR_PER_LAUNCH / (select_ms * 1e-3)
    return {"kernel": "select_tile_kernel", "bound": "alu", "achieved": achieved / 1e9, "peak": peak / 1e9,
            "unit": "G warp-instructions/s", "frac": achieved / peak,
            "peak_kind": f"{N_SM} SMs x {SCHEDULERS_PER_SM} issue slots x {mhz:.0f} MHz",
            "warp_instr_per_pair": NCU_TILE_WARP_INSTR_PER_LAUNCH / NCU_TILE_PAIRS}


def scan_traffic(n_steps: int):
    import hashlib
    path = os.path.join(ROOT, "paper_2509_19086_b200", "csrc", "sja_scan.cuh")
    try:
        sha = hashlib.sha256(open(path, "rb").read()).hexdigest()[:16]
    except OSError:
        return None
    return NCU_SCAN_TRAFFIC_BYTES_PER_STEP * n_steps if sha == NCU_SCAN_SOURCE_SHA else None


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []          # (arrival time, csv line)
        self.t0 = self.t1 = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.perf_counter(), line.strip()))

    def wait_first_sample(self, timeout=10.0):
        t = time.perf_counter()
        while self.proc is not None and not self.lines and time.perf_counter() - t < timeout:
            time.sleep(0.02)

    def mark_begin(self):
        self.t0 = time.perf_counter()

    def mark_end(self):
        self.t1 = time.perf_counter()

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        lines = [ln for (t, ln) in self.lines
                 if self.t0 is None or self.t1 is None or (self.t0 <= t <= self.t1 + 0.15)]
        for ln in lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(smax)) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def _pinned(a: np.ndarray):
    """A pinned torch tensor holding a's bytes and a numpy view of it."""
    import torch
    t = torch.empty(a.nbytes, dtype=torch.uint8).pin_memory()
    v = t.numpy().view(a.dtype).reshape(a.shape)
    v[...] = a
    return t, v


def _to_device(a: np.ndarray, device):
    """Copy a numpy array to the device as a typed torch tensor (u64 -> int64, u32 -> int32 views)."""
    import torch
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint64:
        t = torch.from_numpy(a.view(np.int64))
    elif a.dtype == np.uint8:
        t = torch.from_numpy(a)
    else:
        t = torch.from_numpy(a.view(np.uint8).reshape(-1).view(np.int32))
    return t.to(device, non_blocking=False)


def oracle_rate(prof, gaps, policy, target_s=12.0):
    """Time the CPU oracle (as it stands) on a bounded sample of the workload's gaps."""
    import oracle
    J = prof.n_jobs
    progress = np.zeros(J, np.uint32)
    threads = oracle.num_threads()
    probe = min(gaps.shape[0], max(threads, 8))
    t0 = time.perf_counter()
    oracle.select(prof, progress, prof.ready_ms, gaps[:probe], policy)
    dt = time.perf_counter() - t0
    n = int(min(gaps.shape[0], max(probe, probe * target_s / max(dt, 1e-6))))
    n = max(threads, (n // threads) * threads) if n >= threads else n
    n = min(n, gaps.shape[0])
    t0 = time.perf_counter()
    oracle.select(prof, progress, prof.ready_ms, gaps[:n], policy)
    dt = time.perf_counter() - t0
    return {"value": n * J / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"first {n} of {gaps.shape[0]} gaps x all {J} jobs, naive walk (gcc -O2 -fopenmp), {dt:.2f} s"}


def run_reference(args, spec):
    """The reference arm: the CPU oracle on the host cores, same workload / metric / unit."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    prof = wl.make_profiles(spec, threads=os.cpu_count() or 8)
    gaps = wl.make_gaps(spec)
    import oracle
    J, G = prof.n_jobs, gaps.shape[0]
    progress = np.zeros(J, np.uint32)
    threads = oracle.num_threads()
    # size one step's sample so that warmup + steps stay within a few minutes
    t0 = time.perf_counter()
    probe = min(G, max(threads, 8))
    oracle.select(prof, progress, prof.ready_ms, gaps[:probe], spec.policy)
    per_gap = (time.perf_counter() - t0) / probe
    budget = 120.0 / max(1, args.steps + args.warmup)
    n = int(max(1, min(G, budget / max(per_gap, 1e-9))))
    for _ in range(args.warmup):
        oracle.select(prof, progress, prof.ready_ms, gaps[:n], spec.policy)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        aw = oracle.select(prof, progress, prof.ready_ms, gaps[:n], spec.policy)
        p2, r2 = progress.copy(), prof.ready_ms.copy()
        oracle.commit(p2, r2, gaps[:n], aw)
    dt = time.perf_counter() - t0
    value = args.steps * n * J / dt
    sample = f"per step: first {n} of {G} gaps x all {J} jobs (select + commit), naive walk"
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u32/u64",
        "data": "synthetic", "config": {"workload": spec.name, "jobs": J, "gaps": G, "steps_total": prof.n_steps,
                                        "policy": POLICY_NAMES[spec.policy]},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", type=int, default=2, help="index into the published configuration list")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--flags", type=int, default=0, help="sja_policy.flags (1 = per-pair search kernel, 2 = per-gap merge kernel, 4 = tile kernel at any size)")
    ap.add_argument("--reauction", action="store_true",
                    help="time sja_round_reauction (select + commit repeated for orphaned gaps) instead of one select + commit")
    ap.add_argument("--window-options", action="store_true",
                    help="late start inside a gap and per-job deadlines (ready + 2000..8000 ms): per-pair search path")
    ap.add_argument("--sharded", action="store_true",
                    help="with --gpus N: ONE scheduler over N GPUs (jobs sharded, gaps replicated, one all-gather of a "
                         "32-byte bid per gap and GPU per round) instead of N independent replicas; strong scaling")
    ap.add_argument("--power-caps", action="store_true",
                    help="second resource envelope: a per-step power trace (50 W + 350 W x mem / 80 GiB + noise) loaded "
                         "with every load and a cap of 100..400 W per gap: per-pair search path")
    ap.add_argument("--streaming", action="store_true",
                    help="multi-round workloads only: load once, then every step is one advertise/select/commit round "
                         "with that round's gap batch (use --steps 1000 for the published streaming configuration)")
    ap.add_argument("--jobs", type=int, default=0, help="override the job count (profiling captures)")
    ap.add_argument("--gaps", type=int, default=0, help="override the gap count (profiling captures)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    spec = wl.SPECS[args.workload]
    if args.jobs:
        spec = wl.scaled(spec, n_jobs=args.jobs, name=spec.name + f"-jobs{args.jobs}")
    if args.gaps:
        spec = wl.scaled(spec, n_gaps=args.gaps, name=spec.name + f"-gaps{args.gaps}")

    if args.impl == "reference":
        run_reference(args, spec)
        return
    if args.power_caps:
        args.e2e_steps = 0          # the end-to-end leg moves the four input arrays of the boundary only
    if args.streaming and (spec.n_rounds <= 1 or args.reauction):
        raise SystemExit("--streaming needs a multi-round workload (--workload 4) and no --reauction")

    import torch
    from paper_2509_19086_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=device)

    # replicas: every rank runs an independent scheduler instance on its own seeded workload;
    # sharded: every rank holds a contiguous range of the jobs of the one published workload
    my_spec = spec if args.sharded else replicas.replica_spec(spec, rank)
    prof = wl.make_profiles(my_spec, threads=max(1, (os.cpu_count() or 8) // max(1, world)))
    gaps = wl.make_gaps(my_spec)
    shard_lo = 0
    if args.sharded:
        if args.reauction or args.streaming or args.window_options or args.power_caps:
            raise SystemExit("--sharded times the plain round only")
        from paper_2509_19086_b200 import sharded
        global_jobs = prof.n_jobs
        shard_lo, shard_hi = sharded.shard_bounds(global_jobs, world, rank)
        prof = sharded.shard_profiles(prof, shard_lo, shard_hi)
    J, G, N = prof.n_jobs, int(gaps.shape[0]), prof.n_steps
    pairs = J * G

    stream = torch.cuda.Stream(device=device)
    ctx = binding.Sja(device=local_rank, stream=stream.cuda_stream)

    host_arrays = dict(off=prof.off, d=prof.dur_ms, m=prof.mem_MiB, s=prof.safe_bits, ready=prof.ready_ms)
    if prof.wait_ms is not None:
        host_arrays["wait"] = prof.wait_ms
    if prof.prio is not None:
        host_arrays["prio"] = prof.prio
    pinned_keep, pinned = {}, {}
    for k, a in host_arrays.items():
        pinned_keep[k], pinned[k] = _pinned(a)
    pinned_keep["gaps"], gaps_pinned = _pinned(gaps.view(np.uint8))
    gaps_pinned = gaps_pinned.view(wl.GAP_DTYPE)
    dev = {k: _to_device(a, device) for k, a in host_arrays.items()}
    dev_gaps = _to_device(gaps, device)
    dev_power = dev_caps = None
    if args.power_caps:
        rng = np.random.default_rng(my_spec.seed + 78)
        power = (50 + prof.mem_MiB.astype(np.int64) * 350 // 81920 + rng.integers(0, 120, N)).astype(np.uint32)
        dev_power = _to_device(power, device)
        dev_caps = _to_device(rng.integers(100, 401, G).astype(np.uint32), device)
        del power
    dev_deadline = None
    if args.window_options:
        rng = np.random.default_rng(my_spec.seed + 77)
        deadline = (prof.ready_ms.astype(np.uint64) + rng.integers(2000, 8001, J).astype(np.uint64)).astype(np.uint32)
        dev_deadline = _to_device(deadline, device)
        pinned_keep["deadline"], pinned["deadline"] = _pinned(deadline)
    torch.cuda.synchronize()

    launches = [0]
    one_tile_saving = 3 if G <= 1024 else 0      # a batch of one sort tile is ordered by a single kernel
    round_gaps_dev, round_gaps_pinned = [], []
    if args.streaming:
        # one gap batch per round, resident on the device (and pinned on the host for the end-to-end leg)
        for r in range(max(args.steps, args.warmup, args.e2e_steps)):
            gr = wl.make_gaps(my_spec, r)
            round_gaps_dev.append(_to_device(gr, device))
            if r < args.e2e_steps:
                keep, pin = _pinned(gr.view(np.uint8))
                pinned_keep[f"gaps{r}"] = keep
                round_gaps_pinned.append(pin.view(wl.GAP_DTYPE))
        torch.cuda.synchronize()

    def load_device():
        ctx.load_profiles(dev["off"], dev["d"], dev["m"], dev["s"], dev["ready"],
                          wait_ms=dev.get("wait"), prio=dev.get("prio"))
        if args.window_options:
            ctx.set_window_options(True, dev_deadline)
        if args.power_caps:
            ctx.load_power(dev["off"], dev_power)

    def round_device(r):
        ctx.advertise(round_gaps_dev[r])
        if args.power_caps:
            ctx.advertise_power_caps(dev_caps)
        ctx.select(my_spec.policy, flags=args.flags)
        ctx.commit(want_count=False)
        launches[0] += KERNELS_PER_STEP - 5 - one_tile_saving   # no load: the five load kernels do not run

    def round_e2e(r):
        ctx.advertise(round_gaps_pinned[r])
        aw = ctx.select(my_spec.policy, flags=args.flags, out="host")
        return aw, ctx.commit(want_count=True)

    sched = None
    if args.sharded:
        sched = sharded.ShardedScheduler(ctx, shard_lo, rank, world, dist, device)

    def step_device():
        ctx.load_profiles(dev["off"], dev["d"], dev["m"], dev["s"], dev["ready"],
                          wait_ms=dev.get("wait"), prio=dev.get("prio"))
        if sched is not None:
            # advertise + select on the shard, one all-gather of the bids, fold, commit what this shard won
            sched.round(dev_gaps, my_spec.policy, flags=args.flags)
            launches[0] += KERNELS_PER_STEP - one_tile_saving + 2
            return
        if args.window_options:
            ctx.set_window_options(True, dev_deadline)
        if args.power_caps:
            ctx.load_power(dev["off"], dev_power)
        ctx.advertise(dev_gaps)
        if args.power_caps:
            ctx.advertise_power_caps(dev_caps)
        if args.reauction:
            _, passes = ctx.round_reauction(my_spec.policy, flags=args.flags)
            # 5 load kernels, 4 advertise kernels (1 for a one-tile batch); per pass: select, finalize, 3 commit
            # kernels, orphan compaction
            launches[0] += 9 - one_tile_saving + 6 * passes
        else:
            ctx.select(my_spec.policy, flags=args.flags)
            ctx.commit(want_count=False)
            launches[0] += KERNELS_PER_STEP - one_tile_saving + (1 if args.power_caps else 0)

    def step_e2e():
        ctx.load_profiles(pinned["off"], pinned["d"], pinned["m"], pinned["s"], pinned["ready"],
                          wait_ms=pinned.get("wait"), prio=pinned.get("prio"))
        if sched is not None:
            glob, n = sched.round(gaps_pinned, my_spec.policy, flags=args.flags, want_count=True)
            return glob.cpu(), n
        if args.window_options:
            ctx.set_window_options(True, pinned["deadline"])
        ctx.advertise(gaps_pinned)
        aw = ctx.select(my_spec.policy, flags=args.flags, out="host")
        n = ctx.commit(want_count=True)
        return aw, n

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    with torch.cuda.stream(stream):
        if args.streaming:
            load_device()
            for r in range(args.warmup):
                round_device(r)
            load_device()                      # back to the state before round 0 (untimed)
        else:
            for _ in range(args.warmup):
                step_device()
        n_rows = ctx.scan_size()
        # inside the timed region only the scan kernel (the roofline's kernel) is bracketed by CUDA events;
        # events around every phase cost about 5 % of a step, so that breakdown is taken in a pass of its own below
        ctx.profile_enable(2)
        sampler = ClockSampler(local_rank)
        sampler.start()
        sampler.wait_first_sample()
        barrier()
        sampler.mark_begin()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        launches[0] = 0
        for r in range(args.steps):
            if args.streaming:
                round_device(r)
            else:
                step_device()
        e1.record(stream)
        timed_launches = launches[0]
        barrier()
        sampler.mark_end()
        ms_total = e0.elapsed_time(e1)
        clocks = sampler.stop()
        scan_timing = ctx.profile_read()
        # untimed pass for the per-phase breakdown
        breakdown_steps = min(args.steps, 20)
        if args.streaming:
            load_device()
        ctx.profile_enable(1)
        for r in range(breakdown_steps):
            if args.streaming:
                round_device(r)
            else:
                step_device()
        timing = ctx.profile_read()
        ctx.profile_enable(0)
        if not args.streaming:
            timing["scan_ms"], timing["scan_launches"] = scan_timing["scan_ms"], scan_timing["scan_launches"]

        # end to end: pinned host inputs in, awards + grant count out, every step
        e2e_s = 0.0
        if args.e2e_steps > 0 and args.streaming:
            load_device()
            barrier()
            t0 = time.perf_counter()
            for r in range(args.e2e_steps):
                aw, n_granted = round_e2e(r)
            torch.cuda.synchronize()
            e2e_s = time.perf_counter() - t0
        elif args.e2e_steps > 0:
            step_e2e()
            barrier()
            t0 = time.perf_counter()
            for _ in range(args.e2e_steps):
                aw, n_granted = step_e2e()
            torch.cuda.synchronize()
            e2e_s = time.perf_counter() - t0

    total_pairs, (ms_total, e2e_ms) = replicas.aggregate(pairs, [ms_total, 1e3 * e2e_s], dist, device)
    ms_per_step = ms_total / args.steps
    value = replicas.throughput(total_pairs, args.steps, ms_total)
    e2e_value = replicas.throughput(total_pairs, args.e2e_steps, e2e_ms) if e2e_ms > 0 else None
    h2d = sum(int(a.nbytes) for a in host_arrays.values()) + int(gaps.nbytes) + (4 * J if args.window_options else 0)
    if args.streaming:
        h2d = int(gaps.nbytes)                 # a round moves only its gap batch to the device
    d2h = 24 * G + 4

    peak, peak_kind = measured_peak()
    if args.streaming:
        timing["scan_launches"] = 0            # the scan ran before the timed region
    scan_ms = timing["scan_ms"] / max(1, timing["scan_launches"]) if timing["scan_launches"] else 0.0
    scan_bytes = prof.raw_bytes() + 24 * n_rows
    achieved = scan_bytes / (scan_ms * 1e-3) / 1e9 if scan_ms > 0 else 0.0
    roofline = {
        "kernel": "scan_profiles_kernel", "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
        "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": scan_traffic(N),
        "bytes_per_launch": scan_bytes, "ms_per_launch": scan_ms,
    }
    if args.streaming:
        roofline = None                        # no scan in the timed region; the rounds are bound by instruction issue
    breakdown = {k: timing[k] / breakdown_steps for k in ("prep_ms", "advertise_ms", "select_ms", "commit_ms")}
    breakdown["scan_ms"] = scan_ms
    select_ms = breakdown["select_ms"]

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "strong" if args.sharded else "weak",
        "vs_baseline": None, "dtype": "u32/u64", "data": "synthetic",
        "config": {"workload": my_spec.name if rank == 0 else spec.name, "jobs": J, "gaps": G, "steps_total": N,
                   "boundary_rows": n_rows, "policy": POLICY_NAMES[spec.policy], "parallelism": f"jobs sharded x{world}, one bid all-gather per round" if args.sharded else f"replicas x{world}",
                   "l2": "inputs larger than L2 (profile arrays re-read from HBM every step)"
                   if prof.raw_bytes() > 200e6 else "inputs smaller than L2",
                   "flags": args.flags, "reauction": bool(args.reauction),
                   "window_options": bool(args.window_options), "power_caps": bool(args.power_caps),
                   "jobs_all_ranks": global_jobs if args.sharded else J * world,
                   "streaming": "load once, one advertise/select/commit round per step" if args.streaming else False},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms / max(1, args.e2e_steps), "steps": args.e2e_steps},
        "gpu_launches": timed_launches,
        "roofline": roofline,
        # the instruction count per pair was captured on the large uniform workload only
        "select_roofline": select_roofline(pairs, select_ms, clocks.get("sm_mhz"))
        if spec.index == 2 and not args.flags and not args.reauction and not args.window_options
        and not args.power_caps else None,
        "kernel_ms_per_step": breakdown,
        "select_pairs_per_s": pairs / (select_ms * 1e-3) if select_ms > 0 else None,
        "profile_gb_per_s": prof.raw_bytes() / (scan_ms * 1e-3) / 1e9 if scan_ms > 0 else None,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = oracle_rate(prof, gaps, my_spec.policy)
    ctx.close()
    if rank == 0:
        print(json.dumps(out), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
