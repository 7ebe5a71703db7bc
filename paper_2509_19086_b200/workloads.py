"""Seeded synthetic workloads for the SJA advertise/signal/select round.

This module only draws random inputs (job profiles, job attributes, gap batches).
It contains none of the method's arithmetic: no prefix sums, no feasibility test,
no scoring.  Both the CPU oracle's tests and the CUDA path's tests and benchmark
take their inputs from here, so the two sides always see identical arrays.

The paper (a concept paper, Sections 3.1-3.5, 3.8, 3.9) prescribes no dataset; the
five workloads below follow the distributions of the five published configurations:

* per step ``duration_ms`` ~ U{1..50}, ``mem_MiB`` = clamp(floor(exp(ln 4096 + N(0,1))), 1, 81920),
  safe-boundary bit ~ Bernoulli(p_safe) with the last step of every job safe;
* per job ``ready_ms`` ~ U{0..1000}; ``wait_ms`` ~ U{0..3_600_000}; ``prio`` in {0,1,2}
  with probabilities {0.6, 0.3, 0.1} (larger = more urgent);
* per gap ``slice`` ~ U{0..6}, ``C_MiB`` ~ U{10240, 20480, 40960, 81920}, ``T_ms`` ~ U{100..5000},
  ``start_ms`` ~ U{0..2000} (+ 1000 * round for the streaming workload).

Random streams are counter-based in the sense that every block of jobs and every gap
round owns a generator keyed by ``(seed, stream, index)``; the arrays therefore do not
depend on the number of worker threads used to fill them.
"""
from __future__ import annotations

import dataclasses
import math
from concurrent.futures import ThreadPoolExecutor
from typing import Optional

import numpy as np

BASE_SEED = 250919086

POLICY_EFFICIENCY = 0
POLICY_FAIRNESS = 1
POLICY_SLA = 2

CAPACITIES_MIB = np.array([10240, 20480, 40960, 81920], dtype=np.uint32)
N_SLICES = 7

GAP_DTYPE = np.dtype(
    [("slice", "<u4"), ("start_ms", "<u4"), ("T_ms", "<u4"), ("C_MiB", "<u4")]
)

_STREAM_LEN, _STREAM_STEPS, _STREAM_JOBS, _STREAM_GAPS = 1, 2, 3, 4
_BLOCK_STEPS = 1 << 22


@dataclasses.dataclass(frozen=True)
class WorkloadSpec:
    """Shape of one workload (one entry of the published configuration list)."""

    name: str
    index: int
    n_jobs: int
    n_gaps: int
    policy: int
    n_rounds: int = 1
    fixed_len: Optional[int] = None      # uniform profile length, or None for Zipf
    zipf_s: float = 1.2
    zipf_min: int = 16
    zipf_max: int = 65536
    p_safe: Optional[float] = 0.1        # None: per-job p ~ U[0.01, 0.5]
    with_wait: bool = False
    with_prio: bool = False

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index


SPECS = {
    0: WorkloadSpec("cfg0-tiny", 0, 64, 16, POLICY_EFFICIENCY, fixed_len=256),
    1: WorkloadSpec("cfg1-medium", 1, 4096, 512, POLICY_EFFICIENCY, fixed_len=1024),
    2: WorkloadSpec("cfg2-large-uniform", 2, 65536, 4096, POLICY_FAIRNESS, fixed_len=4096,
                    with_wait=True),
    3: WorkloadSpec("cfg3-heavy-tailed", 3, 262144, 16384, POLICY_SLA, fixed_len=None,
                    p_safe=None, with_prio=True),
    4: WorkloadSpec("cfg4-streaming", 4, 100000, 8192, POLICY_EFFICIENCY, n_rounds=1000,
                    fixed_len=2048),
}


def scaled(spec: WorkloadSpec, **changes) -> WorkloadSpec:
    """A smaller (or otherwise altered) variant of a published configuration."""
    return dataclasses.replace(spec, **changes)


@dataclasses.dataclass
class Profiles:
    """Ragged CSR of per-step job profiles plus per-job attributes."""

    off: np.ndarray        # u64[J+1]
    dur_ms: np.ndarray     # u32[N]
    mem_MiB: np.ndarray    # u32[N]
    safe_bits: np.ndarray  # u32[ceil(N/32)], bit i%32 of word i/32, LSB first
    ready_ms: np.ndarray   # u32[J]
    wait_ms: Optional[np.ndarray]  # u32[J] or None
    prio: Optional[np.ndarray]     # u8[J] or None

    @property
    def n_jobs(self) -> int:
        return int(self.off.shape[0] - 1)

    @property
    def n_steps(self) -> int:
        return int(self.off[-1])

    def raw_bytes(self) -> int:
        """Bytes of profile data one full scan has to read (8 B/step + 1 bit/step)."""
        return 8 * self.n_steps + 4 * int(self.safe_bits.shape[0])


def _rng(seed: int, stream: int, index: int = 0) -> np.random.Generator:
    return np.random.Generator(
        np.random.PCG64(np.random.SeedSequence(entropy=seed, spawn_key=(stream, index)))
    )


def _zipf_lengths(rng: np.random.Generator, n: int, s: float, lo: int, hi: int) -> np.ndarray:
    """P(len = l) proportional to l**-s on the integers lo..hi (inverse-CDF table)."""
    support = np.arange(lo, hi + 1, dtype=np.float64)
    cdf = np.cumsum(support ** (-s))
    cdf /= cdf[-1]
    u = rng.random(n)
    idx = np.searchsorted(cdf, u, side="left")
    return (np.minimum(idx, hi - lo) + lo).astype(np.uint64)


def _job_blocks(off: np.ndarray, block_steps: int) -> list[tuple[int, int]]:
    """Split jobs into consecutive blocks holding about ``block_steps`` steps each.

    Block boundaries depend only on ``off``, so the generated data does not depend on
    how many threads fill the blocks.
    """
    n_jobs = off.shape[0] - 1
    blocks = []
    j0 = 0
    while j0 < n_jobs:
        target = off[j0] + np.uint64(block_steps)
        j1 = int(np.searchsorted(off, target, side="right")) - 1
        j1 = max(j1, j0 + 1)
        j1 = min(j1, n_jobs)
        blocks.append((j0, j1))
        j0 = j1
    return blocks


def make_profiles(spec: WorkloadSpec, threads: int = 8) -> Profiles:
    """Draw the job profiles of ``spec`` (deterministic in ``spec.seed``)."""
    seed = spec.seed
    n_jobs = spec.n_jobs
    if spec.fixed_len is not None:
        lens = np.full(n_jobs, spec.fixed_len, dtype=np.uint64)
    else:
        lens = _zipf_lengths(_rng(seed, _STREAM_LEN), n_jobs, spec.zipf_s,
                             spec.zipf_min, spec.zipf_max)
    off = np.zeros(n_jobs + 1, dtype=np.uint64)
    np.cumsum(lens, out=off[1:])
    n_steps = int(off[-1])

    jr = _rng(seed, _STREAM_JOBS)
    ready = jr.integers(0, 1001, size=n_jobs, dtype=np.uint32)
    wait = jr.integers(0, 3_600_001, size=n_jobs, dtype=np.uint32) if spec.with_wait else None
    prio = None
    if spec.with_prio:
        prio = jr.choice(np.array([0, 1, 2], dtype=np.uint8), size=n_jobs,
                         p=[0.6, 0.3, 0.1]).astype(np.uint8)
    if spec.p_safe is None:
        p_job = jr.uniform(0.01, 0.5, size=n_jobs)
    else:
        p_job = None

    dur = np.empty(n_steps, dtype=np.uint32)
    mem = np.empty(n_steps, dtype=np.uint32)
    safe = np.empty(n_steps, dtype=np.uint8)
    ln_mu = math.log(4096.0)
    blocks = _job_blocks(off, _BLOCK_STEPS)

    def fill(bi: int) -> None:
        j0, j1 = blocks[bi]
        a, b = int(off[j0]), int(off[j1])
        n = b - a
        if n == 0:
            return
        rng = _rng(seed, _STREAM_STEPS, bi)
        dur[a:b] = rng.integers(1, 51, size=n, dtype=np.uint32)
        z = rng.standard_normal(n)
        np.add(z, ln_mu, out=z)
        np.exp(z, out=z)
        np.floor(z, out=z)
        np.clip(z, 1.0, 81920.0, out=z)
        mem[a:b] = z.astype(np.uint32)
        u = rng.random(n, dtype=np.float32)
        if p_job is None:
            safe[a:b] = u < np.float32(spec.p_safe)
        else:
            reps = (off[j0 + 1:j1 + 1] - off[j0:j1]).astype(np.int64)
            safe[a:b] = u < np.repeat(p_job[j0:j1], reps).astype(np.float32)

    if threads > 1 and len(blocks) > 1:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(fill, range(len(blocks))))
    else:
        for bi in range(len(blocks)):
            fill(bi)

    nonempty = lens > 0
    last = (off[1:][nonempty] - np.uint64(1)).astype(np.int64)
    safe[last] = 1
    bits = pack_safe_bits(safe)
    return Profiles(off, dur, mem, bits, ready, wait, prio)


def pack_safe_bits(safe: np.ndarray) -> np.ndarray:
    """Pack a 0/1 array into u32 words, bit ``i % 32`` of word ``i // 32`` (LSB first)."""
    n = int(safe.shape[0])
    n_words = (n + 31) // 32
    packed = np.packbits(safe.astype(np.uint8, copy=False), bitorder="little")
    out = np.zeros(n_words * 4, dtype=np.uint8)
    out[: packed.shape[0]] = packed
    return out.view("<u4")


def unpack_safe_bits(bits: np.ndarray, n: int) -> np.ndarray:
    """Inverse of :func:`pack_safe_bits` (layout helper, used by tests)."""
    return np.unpackbits(bits.view(np.uint8), bitorder="little")[:n]


def make_gaps(spec: WorkloadSpec, round_index: int = 0, n_gaps: Optional[int] = None) -> np.ndarray:
    """Draw the gap batch advertised in round ``round_index`` (structured ``GAP_DTYPE``)."""
    g = spec.n_gaps if n_gaps is None else n_gaps
    rng = _rng(spec.seed, _STREAM_GAPS, round_index)
    gaps = np.empty(g, dtype=GAP_DTYPE)
    gaps["slice"] = rng.integers(0, N_SLICES, size=g, dtype=np.uint32)
    gaps["C_MiB"] = CAPACITIES_MIB[rng.integers(0, 4, size=g)]
    gaps["T_ms"] = rng.integers(100, 5001, size=g, dtype=np.uint32)
    base = 1000 * round_index if spec.n_rounds > 1 else 0
    gaps["start_ms"] = rng.integers(0, 2001, size=g, dtype=np.uint32) + np.uint32(base)
    return gaps


def checksum64(a: np.ndarray) -> int:
    """Order-sensitive 64-bit checksum of an array's bytes (for reproducibility logs)."""
    b = np.ascontiguousarray(a).view(np.uint8)
    pad = (-b.shape[0]) % 8
    if pad:
        b = np.concatenate([b, np.zeros(pad, dtype=np.uint8)])
    w = b.view("<u8")
    idx = np.arange(1, w.shape[0] + 1, dtype=np.uint64)
    with np.errstate(over="ignore"):
        mixed = (w ^ (idx * np.uint64(0x9E3779B97F4A7C15))) * np.uint64(0xBF58476D1CE4E5B9)
        return int(np.bitwise_xor.reduce(mixed) ^ np.add.reduce(mixed))


def _main() -> None:
    """Print the reproducibility table: per configuration the step count and array checksums."""
    import argparse
    import time

    ap = argparse.ArgumentParser(description="checksums of the seeded synthetic workloads")
    ap.add_argument("configs", nargs="*", type=int, default=[0, 1, 2, 3, 4])
    ap.add_argument("--threads", type=int, default=8)
    args = ap.parse_args()
    print("| cfg | seed | jobs | N steps | checksum(dur) | checksum(mem) | checksum(safe) | checksum(ready) | checksum(gaps r0) |")
    print("|---|---|---|---|---|---|---|---|---|")
    for c in args.configs:
        spec = SPECS[c]
        t0 = time.time()
        prof = make_profiles(spec, threads=args.threads)
        gaps = make_gaps(spec)
        cs = [checksum64(a) for a in (prof.dur_ms, prof.mem_MiB, prof.safe_bits, prof.ready_ms, gaps)]
        print(f"| {c} | {spec.seed} | {prof.n_jobs} | {prof.n_steps} | " + " | ".join(f"{x:016x}" for x in cs)
              + f" | <!-- {time.time() - t0:.1f} s -->")


if __name__ == "__main__":
    _main()
