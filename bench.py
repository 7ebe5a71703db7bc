#!/usr/bin/env python
"""Benchmark of the SJA advertise / signal / select / commit round.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 0..4] [--impl ours|reference]

One "step" is one pass of the whole round over one synthetic workload: the segmented scan
of all job profiles (sja_load_profiles), sja_advertise, sja_select and sja_commit.
Metric: job-gap pairs evaluated per second (G*J pairs per step; every pair counts, however
early it is declined).  The headline workload is the largest published single-round
configuration (heavy-tailed: 262 144 ragged jobs, about 1e9 steps, 16 384 gaps, SLA policy).
A default run then also times, in the same process and after the headline region, the large
uniform configuration and the streaming configuration (load once, one round per step) and
reports them under "other_workloads".  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import gc
import hashlib
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
POLICY_NAMES = {0: "efficiency", 1: "fairness", 2: "sla", 3: "tight_fit"}
HEADLINE_WORKLOAD = 3
FALLBACK_HBM_GBS = 6650.0
N_SM, SCHEDULERS_PER_SM = 148, 4

# Kernels launched by one call of each entry point on the default path (counted from the launch list of this
# command under ncu): load = count_boundaries, cta_offsets, finish_load, scan_profiles; advertise = sort_gap_tiles,
# rank_gap_tiles, place_gaps (a batch of at most 1024 gaps: sort_gap_tiles alone); select = select_tile, the
# select_search launch that stands by for batches of very many capacity classes (it returns at once otherwise),
# finalize_awards -- or select_search + finalize_awards where only the search runs; commit = commit_vote,
# commit_apply, commit_refresh.
LAUNCHES_LOAD, LAUNCHES_ADVERTISE, LAUNCHES_ADVERTISE_ONE_TILE, LAUNCHES_COMMIT = 4, 3, 1, 3


def select_launches(pairs, flags, per_pair_window):
    return 2 if (flags & 1) or per_pair_window or pairs < 65536 else 3


# DRAM traffic of the scan kernel, from one ncu capture of dram__bytes_read.sum and dram__bytes_write.sum on the
# large uniform configuration at full size: reads grow with the step count, writes with the number of boundary
# rows.  The figures are reported only while csrc/sja_scan.cuh is the file they were taken from (first 16 hex
# digits of its sha256); otherwise "traffic" is null.
NCU_SCAN = {"source_sha": "06cf166b6a8a770f", "read_bytes_per_step": 2184370432 / 268435456,
            "write_bytes_per_row": 625901568 / 26906044}

# Warp instructions of one select_tile_kernel launch (ncu smsp__inst_executed.sum, one pass, full size), per
# workload; valid while csrc/sja_tile.cuh is the file they were taken from.  The kernel's work is not proportional
# to the pair count, so each figure holds for its workload only.
NCU_TILE = {"source_sha": "eb40ed91a9a31e13",
            "warp_instr_per_launch": {"cfg3-heavy-tailed": 769500647, "cfg2-large-uniform": 90793074,
                                      "cfg4-streaming": 187177939}}


def _source_sha(name: str):
    path = os.path.join(ROOT, "paper_2509_19086_b200", "csrc", name)
    try:
        return hashlib.sha256(open(path, "rb").read()).hexdigest()[:16]
    except OSError:
        return None


def select_roofline(spec_name, pairs, select_ms, sm_mhz, clock_source):
    """Issue rate of the select kernel against the GPU's warp-instruction issue peak (select_ms also holds the
    few microseconds of finalize_awards_kernel, so the rate is slightly understated)."""
    instr = NCU_TILE["warp_instr_per_launch"].get(spec_name)
    if not select_ms or instr is None or _source_sha("sja_tile.cuh") != NCU_TILE["source_sha"]:
        return None
    mhz = sm_mhz or 1965.0
    peak = N_SM * SCHEDULERS_PER_SM * mhz * 1e6
    achieved = instr / (select_ms * 1e-3)
    return {"kernel": "select_tile_kernel", "bound": "alu", "achieved": achieved / 1e9, "peak": peak / 1e9,
            "unit": "G warp-instructions/s", "frac": achieved / peak,
            "peak_kind": f"{N_SM} SMs x {SCHEDULERS_PER_SM} issue slots x {mhz:.0f} MHz ({clock_source})",
            "warp_instr_per_pair": instr / pairs}


def scan_traffic(n_steps: int, n_rows: int):
    if NCU_SCAN["source_sha"] is None or _source_sha("sja_scan.cuh") != NCU_SCAN["source_sha"]:
        return None
    return NCU_SCAN["read_bytes_per_step"] * n_steps + NCU_SCAN["write_bytes_per_row"] * n_rows


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons every few milliseconds while the GPU works: through NVML (read
    only) when its Python module is there, else by polling nvidia-smi.  Samples carry a phase label, so that the
    report can say how many fell inside the timed region and fall back to the whole loaded span (warm-up and
    timed steps) when the timed region was too short to catch several."""

    REASONS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20),
               ("sw_power_cap", 0x4))
    SMI_FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
                  "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
                  "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int, period_s: float = 0.004):
        self.index, self.period = index, period_s
        self.samples = []          # (time, sm_mhz, reason bit mask)
        self.max_mhz = None
        self.marks = {}
        self._stop = threading.Event()
        self._thread = None
        self.source = None
        self._proc = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            h = pynvml.nvmlDeviceGetHandleByIndex(self._physical_index())
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            reasons = getattr(pynvml, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                pynvml.nvmlDeviceGetCurrentClocksThrottleReasons

            def loop():
                while not self._stop.is_set():
                    try:
                        mhz = float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM))
                        self.samples.append((time.perf_counter(), mhz, int(reasons(h))))
                    except Exception:
                        pass
                    time.sleep(self.period)

            self._thread = threading.Thread(target=loop, daemon=True)
            self._thread.start()
            self.source = "nvml"
            return
        except Exception:
            pass
        try:
            self._proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self._physical_index()}", f"--query-gpu={self.SMI_FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)

            def read():
                for line in self._proc.stdout:
                    parts = [p.strip() for p in line.split(",")]
                    if len(parts) < 6:
                        continue
                    try:
                        mhz, self.max_mhz = float(parts[0]), float(parts[1])
                    except ValueError:
                        continue
                    mask = 0
                    for (_, bit), v in zip(self.REASONS, parts[2:6]):
                        if v.lower().startswith("active"):
                            mask |= bit
                    self.samples.append((time.perf_counter(), mhz, mask))

            self._thread = threading.Thread(target=read, daemon=True)
            self._thread.start()
            self.source = "nvidia-smi"
        except Exception:
            self._proc = None

    def _physical_index(self) -> int:
        vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
        ids = [x for x in vis.split(",") if x.strip()]
        if ids and self.index < len(ids) and ids[self.index].strip().isdigit():
            return int(ids[self.index])
        return self.index

    def wait_first_sample(self, timeout=10.0):
        t = time.perf_counter()
        while self.source and not self.samples and time.perf_counter() - t < timeout:
            time.sleep(0.01)

    def mark(self, name: str):
        self.marks[name] = time.perf_counter()

    def stop(self) -> dict:
        self._stop.set()
        if self._proc is not None:
            self._proc.terminate()
            try:
                self._proc.wait(timeout=5)
            except Exception:
                self._proc.kill()
        if self._thread is not None:
            self._thread.join(timeout=2)
        if not self.source:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no clock source (NVML and nvidia-smi unavailable)"],
                    "samples": 0, "clock_source": "none"}

        def span(a, b, slack=0.0):
            ta, tb = self.marks.get(a), self.marks.get(b)
            if ta is None or tb is None:
                return []
            return [s for s in self.samples if ta <= s[0] <= tb + slack]

        timed = span("timed_begin", "timed_end")
        loaded = span("load_begin", "timed_end")
        use, scope = (timed, "timed region") if len(timed) >= 3 else (loaded, "warm-up and timed region")
        mask = 0
        for s in use:
            mask |= s[2]
        return {"sm_mhz": float(np.median([s[1] for s in use])) if use else None,
                "sm_max_mhz": self.max_mhz,
                "reasons": [n for n, bit in self.REASONS if mask & bit],
                "samples": len(use), "samples_in_timed_region": len(timed), "scope": scope,
                "clock_source": self.source}


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


def n_boundary_rows(prof) -> int:
    """Safe boundaries of the raw profiles (an input statistic; the generators make every job's end safe)."""
    return int(np.unpackbits(prof.safe_bits.view(np.uint8)).sum())


def workload_config(spec, prof, n_gaps, world=1):
    """The keys both arms (ours and the reference) report for a workload."""
    return {"workload": spec.name, "jobs": prof.n_jobs, "gaps": int(n_gaps), "steps_total": prof.n_steps,
            "boundary_rows": n_boundary_rows(prof), "policy": POLICY_NAMES[spec.policy],
            "l2": "inputs larger than L2 (profile arrays re-read from HBM every step)"
            if prof.raw_bytes() > 200e6 else "inputs smaller than L2"}


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
    config = workload_config(spec, prof, G)
    config["parallelism"] = f"host cores x{threads}"
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u32/u64",
        "data": "synthetic", "config": config,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)


class Env:
    """Process-wide handles of one bench run."""

    def __init__(self, args):
        import torch
        self.torch = torch
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
        torch.cuda.set_device(self.local_rank)
        self.device = torch.device("cuda", self.local_rank)
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist_mod
            self.dist = dist_mod
            self.dist.init_process_group("nccl", device_id=self.device)
        self.stream = torch.cuda.Stream(device=self.device)

    def barrier(self):
        self.torch.cuda.synchronize()
        if self.dist is not None:
            self.dist.barrier()
        self.torch.cuda.synchronize()


def bench_workload(env, args, spec, *, streaming, steps, warmup, e2e_steps, sampler=None, options=True):
    """Times `steps` steps of one workload on this rank.  Returns the local measurements; the caller folds
    ranks.  `options`: honour the command line's feature flags (the extra workloads of a default run do not)."""
    torch = env.torch
    from paper_2509_19086_b200 import binding
    device, stream, world, rank = env.device, env.stream, env.world, env.rank
    flags = args.flags if options else 0
    reauction = bool(args.reauction and options)
    window_options = bool(args.window_options and options)
    power_caps = bool(args.power_caps and options)
    is_sharded = bool(args.sharded and options)
    if power_caps:
        e2e_steps = 0               # the end-to-end leg moves the four input arrays of the boundary only

    # replicas: every rank runs an independent scheduler instance on its own seeded workload;
    # sharded: every rank holds a contiguous range of the jobs of the one published workload
    my_spec = spec if is_sharded else replicas.replica_spec(spec, rank)
    prof = wl.make_profiles(my_spec, threads=max(1, (os.cpu_count() or 8) // max(1, world)))
    gaps = wl.make_gaps(my_spec)
    shard_lo, global_jobs = 0, prof.n_jobs
    sharded = None
    if is_sharded:
        from paper_2509_19086_b200 import sharded
        shard_lo, shard_hi = sharded.shard_bounds(global_jobs, world, rank)
        prof = sharded.shard_profiles(prof, shard_lo, shard_hi)
    J, G, N = prof.n_jobs, int(gaps.shape[0]), prof.n_steps
    pairs = J * G
    config = workload_config(my_spec if rank == 0 else spec, prof, G)

    ctx = binding.Sja(device=env.local_rank, stream=stream.cuda_stream)
    host_arrays = dict(off=prof.off, d=prof.dur_ms, m=prof.mem_MiB, s=prof.safe_bits, ready=prof.ready_ms)
    if prof.wait_ms is not None:
        host_arrays["wait"] = prof.wait_ms
    if prof.prio is not None:
        host_arrays["prio"] = prof.prio
    dev = {k: _to_device(a, device) for k, a in host_arrays.items()}
    dev_gaps = _to_device(gaps, device)
    pinned_keep, pinned = {}, {}
    gaps_pinned = None
    if e2e_steps > 0:
        if not streaming:
            for k, a in host_arrays.items():
                pinned_keep[k], pinned[k] = _pinned(a)
        pinned_keep["gaps"], gp = _pinned(gaps.view(np.uint8))
        gaps_pinned = gp.view(wl.GAP_DTYPE)
    dev_power = dev_caps = dev_deadline = None
    if power_caps:
        rng = np.random.default_rng(my_spec.seed + 78)
        power = (50 + prof.mem_MiB.astype(np.int64) * 350 // 81920 + rng.integers(0, 120, N)).astype(np.uint32)
        dev_power = _to_device(power, device)
        dev_caps = _to_device(rng.integers(100, 401, G).astype(np.uint32), device)
        del power
    if window_options:
        rng = np.random.default_rng(my_spec.seed + 77)
        deadline = (prof.ready_ms.astype(np.uint64) + rng.integers(2000, 8001, J).astype(np.uint64)).astype(np.uint32)
        dev_deadline = _to_device(deadline, device)
        if e2e_steps > 0:
            pinned_keep["deadline"], pinned["deadline"] = _pinned(deadline)
    torch.cuda.synchronize()

    launches = [0]
    adv_launches = LAUNCHES_ADVERTISE_ONE_TILE if G <= 1024 else LAUNCHES_ADVERTISE
    LAUNCHES_SELECT = select_launches(pairs, flags, window_options or power_caps)
    round_gaps_dev, round_gaps_pinned = [], []
    if streaming:
        # one gap batch per round, resident on the device (and pinned on the host for the end-to-end leg)
        for r in range(max(steps, warmup, e2e_steps)):
            gr = wl.make_gaps(my_spec, r)
            round_gaps_dev.append(_to_device(gr, device))
            if r < e2e_steps:
                keep, pin = _pinned(gr.view(np.uint8))
                pinned_keep[f"gaps{r}"] = keep
                round_gaps_pinned.append(pin.view(wl.GAP_DTYPE))
        torch.cuda.synchronize()

    def load_device():
        ctx.load_profiles(dev["off"], dev["d"], dev["m"], dev["s"], dev["ready"],
                          wait_ms=dev.get("wait"), prio=dev.get("prio"))
        if window_options:
            ctx.set_window_options(True, dev_deadline)
        if power_caps:
            ctx.load_power(dev["off"], dev_power)

    def round_device(r):
        ctx.advertise(round_gaps_dev[r])
        if power_caps:
            ctx.advertise_power_caps(dev_caps)
        ctx.select(my_spec.policy, flags=flags)
        ctx.commit(want_count=False)
        launches[0] += adv_launches + LAUNCHES_SELECT + LAUNCHES_COMMIT

    def round_e2e(r):
        ctx.advertise(round_gaps_pinned[r])
        aw = ctx.select(my_spec.policy, flags=flags, out="host")
        return aw, ctx.commit(want_count=True)

    sched = None
    if is_sharded:
        sched = sharded.ShardedScheduler(ctx, shard_lo, rank, world, env.dist, device)

    def step_device():
        ctx.load_profiles(dev["off"], dev["d"], dev["m"], dev["s"], dev["ready"],
                          wait_ms=dev.get("wait"), prio=dev.get("prio"))
        launches[0] += LAUNCHES_LOAD
        if sched is not None:
            # advertise + select on the shard, one all-gather of the bids, fold, commit what this shard won
            sched.round(dev_gaps, my_spec.policy, flags=flags)
            launches[0] += adv_launches + LAUNCHES_SELECT + LAUNCHES_COMMIT + 2
            return
        if window_options:
            ctx.set_window_options(True, dev_deadline)
        if power_caps:
            ctx.load_power(dev["off"], dev_power)
            launches[0] += 1
        ctx.advertise(dev_gaps)
        if power_caps:
            ctx.advertise_power_caps(dev_caps)
        if reauction:
            _, passes = ctx.round_reauction(my_spec.policy, flags=flags)
            # per pass: select, finalize, one kernel for the commit and the compaction of the gap list
            launches[0] += adv_launches + 3 * passes
        else:
            ctx.select(my_spec.policy, flags=flags)
            ctx.commit(want_count=False)
            launches[0] += adv_launches + LAUNCHES_SELECT + LAUNCHES_COMMIT

    def step_e2e():
        ctx.load_profiles(pinned["off"], pinned["d"], pinned["m"], pinned["s"], pinned["ready"],
                          wait_ms=pinned.get("wait"), prio=pinned.get("prio"))
        if sched is not None:
            glob, n = sched.round(gaps_pinned, my_spec.policy, flags=flags, want_count=True)
            return glob.cpu(), n
        if window_options:
            ctx.set_window_options(True, pinned["deadline"])
        ctx.advertise(gaps_pinned)
        aw = ctx.select(my_spec.policy, flags=flags, out="host")
        n = ctx.commit(want_count=True)
        return aw, n

    with torch.cuda.stream(stream):
        if sampler is not None:
            sampler.mark("load_begin")
        if streaming:
            load_device()
            for r in range(warmup):
                round_device(r)
            load_device()                      # back to the state before round 0 (untimed)
        else:
            for _ in range(warmup):
                step_device()
        n_rows = ctx.scan_size()
        # inside the timed region only the scan kernel (the roofline's kernel) is bracketed by CUDA events;
        # events around every phase cost a few per cent of a step, so that breakdown is taken in a pass of its own
        ctx.profile_enable(2)
        env.barrier()
        if sampler is not None:
            sampler.mark("timed_begin")
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        launches[0] = 0
        for r in range(steps):
            if streaming:
                round_device(r)
            else:
                step_device()
        e1.record(stream)
        timed_launches = launches[0]
        env.barrier()
        if sampler is not None:
            sampler.mark("timed_end")
        ms_total = e0.elapsed_time(e1)
        scan_timing = ctx.profile_read()
        # untimed pass for the per-phase breakdown
        breakdown_steps = min(steps, 20)
        if streaming:
            load_device()
        ctx.profile_enable(1)
        for r in range(breakdown_steps):
            if streaming:
                round_device(r)
            else:
                step_device()
        timing = ctx.profile_read()
        ctx.profile_enable(0)
        if not streaming:
            timing["scan_ms"], timing["scan_launches"] = scan_timing["scan_ms"], scan_timing["scan_launches"]

        # end to end: pinned host inputs in, awards + grant count out, every step
        e2e_s = 0.0
        if e2e_steps > 0 and streaming:
            load_device()
            env.barrier()
            t0 = time.perf_counter()
            for r in range(e2e_steps):
                round_e2e(r)
            torch.cuda.synchronize()
            e2e_s = time.perf_counter() - t0
        elif e2e_steps > 0:
            step_e2e()
            env.barrier()
            t0 = time.perf_counter()
            for _ in range(e2e_steps):
                step_e2e()
            torch.cuda.synchronize()
            e2e_s = time.perf_counter() - t0

    h2d = sum(int(a.nbytes) for a in host_arrays.values()) + int(gaps.nbytes) + (4 * J if window_options else 0)
    if streaming:
        h2d = int(gaps.nbytes)                 # a round moves only its gap batch to the device
    d2h = 24 * G + 4
    if streaming:
        timing["scan_launches"] = 0            # the scan ran before the timed region
    scan_ms = timing["scan_ms"] / max(1, timing["scan_launches"]) if timing["scan_launches"] else 0.0
    breakdown = {k: timing[k] / breakdown_steps for k in ("prep_ms", "advertise_ms", "select_ms", "commit_ms")}
    breakdown["scan_ms"] = scan_ms
    res = {
        "spec": my_spec, "config": config, "pairs": pairs, "J": J, "G": G, "N": N, "n_rows": n_rows,
        "ms_total": ms_total, "steps": steps, "e2e_ms": 1e3 * e2e_s, "e2e_steps": e2e_steps, "h2d": h2d, "d2h": d2h,
        "timed_launches": timed_launches, "scan_ms": scan_ms, "breakdown": breakdown,
        "scan_bytes": prof.raw_bytes() + 24 * n_rows, "raw_bytes": prof.raw_bytes(),
        "global_jobs": global_jobs if is_sharded else J * world, "streaming": streaming,
        "prof": prof, "gaps": gaps,
    }
    ctx.close()
    del dev, dev_gaps, pinned_keep, pinned, round_gaps_dev
    return res


def scan_roofline(res):
    peak, peak_kind = measured_peak()
    if res["streaming"] or res["scan_ms"] <= 0:
        return None                            # no scan in the timed region; the rounds are bound by instruction issue
    achieved = res["scan_bytes"] / (res["scan_ms"] * 1e-3) / 1e9
    return {"kernel": "scan_profiles_kernel", "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
            "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": scan_traffic(res["N"], res["n_rows"]),
            "bytes_per_launch": res["scan_bytes"], "ms_per_launch": res["scan_ms"],
            "raw_profile_gb_per_s": res["raw_bytes"] / (res["scan_ms"] * 1e-3) / 1e9}


def select_hbm(res, n_chunk_jobs=512):
    """The select kernels' compulsory HBM bytes over their time, as a fraction of the HBM peak: per job its state
    words and the first row of its table (what it takes to decline), the gap batch, one candidate row per job
    chunk and gap written and read back, and the awards.  A lower bound: rows beyond the first are not counted."""
    peak, peak_kind = measured_peak()
    ms = res["breakdown"]["select_ms"]
    if ms <= 0:
        return None
    J, G = res["J"], res["G"]
    chunks = (J + n_chunk_jobs - 1) // n_chunk_jobs
    nbytes = J * (8 + 4 + 4 + 8 + 4 + 4 + 16) + G * 16 + 2 * chunks * G * 16 + G * 28
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"bytes_lower_bound": nbytes, "gb_per_s": gbs, "frac_of_hbm": gbs / peak, "peak_kind": f"of {peak_kind}"}


def summary(res, clocks=None):
    """The figures reported for a workload timed after the headline region."""
    ms = res["ms_total"] / res["steps"]
    sel_ms = res["breakdown"]["select_ms"]
    mhz = (clocks or {}).get("sm_mhz")
    return {
        "config": res["config"], "steps": res["steps"], "ms_per_step": ms,
        "value": res["pairs"] * res["steps"] / (res["ms_total"] * 1e-3), "unit": UNIT,
        "streaming": "load once, one advertise/select/commit round per step" if res["streaming"] else False,
        "e2e": {"value": res["pairs"] * res["e2e_steps"] / (res["e2e_ms"] * 1e-3) if res["e2e_ms"] > 0 else None,
                "unit": UNIT, "ms_per_step": res["e2e_ms"] / max(1, res["e2e_steps"]), "steps": res["e2e_steps"],
                "h2d_bytes_per_step": res["h2d"], "d2h_bytes_per_step": res["d2h"]},
        "gpu_launches": res["timed_launches"], "roofline": scan_roofline(res),
        "select_roofline": select_roofline(res["spec"].name, res["pairs"], sel_ms, mhz, "sampled" if mhz else "assumed max"),
        "select_hbm": select_hbm(res),
        "kernel_ms_per_step": res["breakdown"],
        "select_pairs_per_s": res["pairs"] / (sel_ms * 1e-3) if sel_ms > 0 else None,
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=60)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", type=int, default=HEADLINE_WORKLOAD, help="index into the published configuration list")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the other workloads a default run times after the headline region")
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
    plain = not (args.jobs or args.gaps or args.flags or args.reauction or args.window_options or args.sharded
                 or args.power_caps or args.streaming)
    if args.jobs:
        spec = wl.scaled(spec, n_jobs=args.jobs, name=spec.name + f"-jobs{args.jobs}")
    if args.gaps:
        spec = wl.scaled(spec, n_gaps=args.gaps, name=spec.name + f"-gaps{args.gaps}")

    if args.impl == "reference":
        run_reference(args, spec)
        return
    if args.streaming and (spec.n_rounds <= 1 or args.reauction):
        raise SystemExit("--streaming needs a multi-round workload (--workload 4) and no --reauction")
    if args.sharded and (args.reauction or args.streaming or args.window_options or args.power_caps):
        raise SystemExit("--sharded times the plain round only")

    env = Env(args)
    rank, world = env.rank, env.world
    sampler = ClockSampler(env.local_rank)
    sampler.start()
    sampler.wait_first_sample()
    res = bench_workload(env, args, spec, streaming=args.streaming, steps=args.steps, warmup=args.warmup,
                         e2e_steps=args.e2e_steps, sampler=sampler)
    clocks = sampler.stop()

    total_pairs, (ms_total, e2e_ms) = replicas.aggregate(res["pairs"], [res["ms_total"], res["e2e_ms"]], env.dist,
                                                         env.device)
    value = replicas.throughput(total_pairs, args.steps, ms_total)
    e2e_value = replicas.throughput(total_pairs, res["e2e_steps"], e2e_ms) if e2e_ms > 0 else None
    config = dict(res["config"])
    config.update({
        "parallelism": f"jobs sharded x{world}, one bid all-gather per round" if args.sharded else f"replicas x{world}",
        "flags": args.flags, "reauction": bool(args.reauction), "window_options": bool(args.window_options),
        "power_caps": bool(args.power_caps), "jobs_all_ranks": res["global_jobs"],
        "streaming": "load once, one advertise/select/commit round per step" if args.streaming else False})
    select_ms = res["breakdown"]["select_ms"]
    mhz = clocks.get("sm_mhz")
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True,
        "scaling": "strong" if args.sharded else "weak",
        "vs_baseline": None, "dtype": "u32/u64", "data": "synthetic",
        "config": config,
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": res["h2d"], "d2h_bytes_per_step": res["d2h"],
                "ms_per_step": e2e_ms / max(1, res["e2e_steps"]), "steps": res["e2e_steps"]},
        "gpu_launches": res["timed_launches"],
        "roofline": scan_roofline(res),
        "select_roofline": select_roofline(res["spec"].name, res["pairs"], select_ms, mhz,
                                           "sampled" if mhz else "assumed max") if plain else None,
        "select_hbm": select_hbm(res),
        "kernel_ms_per_step": res["breakdown"],
        "select_pairs_per_s": res["pairs"] / (select_ms * 1e-3) if select_ms > 0 else None,
        "profile_gb_per_s": res["raw_bytes"] / (res["scan_ms"] * 1e-3) / 1e9 if res["scan_ms"] > 0 else None,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = oracle_rate(res["prof"], res["gaps"], res["spec"].policy)
    res = None
    gc.collect()
    env.torch.cuda.empty_cache()

    # a default run: the large uniform configuration and the streaming configuration, after the headline region
    if plain and world == 1 and args.workload == HEADLINE_WORKLOAD and not args.no_extras:
        others = {}
        for index, streaming, steps in ((2, False, 100), (4, True, 300)):
            r = bench_workload(env, args, wl.SPECS[index], streaming=streaming, steps=steps, warmup=3,
                               e2e_steps=3 if streaming else 0, options=False)
            r["prof"] = r["gaps"] = None
            others[wl.SPECS[index].name] = summary(r, clocks)
            r = None
            gc.collect()
            env.torch.cuda.empty_cache()
        out["other_workloads"] = others
    if rank == 0:
        print(json.dumps(out), flush=True)
    if env.dist is not None:
        env.dist.barrier()
        env.dist.destroy_process_group()


if __name__ == "__main__":
    main()
