#!/usr/bin/env python
"""Writes tests/golden/trajectory_cfg4.json and tests/golden/trajectory_cfg3.json.

    python tests/golden/make_trajectories.py [cfg4] [cfg3] [--threads N]

Every stored value comes from the CPU oracles (oracle/trajectory.py); nothing here touches the CUDA path.
The inputs are the seeded synthetic workloads of the two published configurations.  On 8 host cores the
streaming configuration takes about an hour, the heavy-tailed one a few minutes.
"""
import argparse
import json
import os
import sys
import time

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import trajectory  # noqa: E402
from paper_2509_19086_b200 import workloads as wl  # noqa: E402


def _log(msg):
    print(time.strftime("%H:%M:%S"), msg, flush=True)


def _write(name, doc):
    path = os.path.join(HERE, name)
    with open(path + ".tmp", "w") as f:
        json.dump(doc, f, separators=(",", ":"))
        f.write("\n")
    os.replace(path + ".tmp", path)
    _log(f"wrote {path}")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("which", nargs="*", default=["cfg3", "cfg4"])
    ap.add_argument("--threads", type=int, default=os.cpu_count() or 8, help="threads of the input generator")
    args = ap.parse_args()
    for name in args.which:
        index = {"cfg3": 3, "cfg4": 4}[name]
        spec = wl.SPECS[index]
        _log(f"{spec.name}: generating inputs")
        prof = wl.make_profiles(spec, threads=args.threads)
        head = {"workload": spec.name, "seed": spec.seed, "jobs": prof.n_jobs, "steps_total": prof.n_steps,
                "gaps_per_round": spec.n_gaps,
                "source": "oracle/trajectory.py via tests/golden/make_trajectories.py (CPU oracles only)"}
        if index == 4:
            doc = trajectory.streaming_trajectory(prof, lambda r: wl.make_gaps(spec, r), spec.n_rounds,
                                                  spec.policy, log=_log)
        else:
            doc = trajectory.single_round(prof, wl.make_gaps(spec), spec.policy, log=_log)
        head.update(doc)
        _write(f"trajectory_{name}.json", head)


if __name__ == "__main__":
    main()
