"""CPU-only checks of the C-ABI boundary: the library loads and exports what the header declares."""
import ctypes
import os
import re

import numpy as np

from paper_2509_19086_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "sja.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sja_[a-z_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build_library()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    declared = _declared_symbols()
    assert "sja_load_profiles" in declared and "sja_select" in declared
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in include/sja.h but not exported"
    assert sorted(binding.EXPORTS) == declared


def test_struct_layouts_match_header():
    assert binding.GAP_DTYPE.itemsize == 16
    assert binding.AWARD_DTYPE.itemsize == 24
    assert binding.AWARD_DTYPE.fields["score"][1] == 16
    assert ctypes.sizeof(binding.SjaPolicy) == 8
    assert ctypes.sizeof(binding.SjaTiming) == 40
    from paper_2509_19086_b200 import workloads as wl
    assert wl.GAP_DTYPE == binding.GAP_DTYPE


def test_null_context_calls_are_rejected_without_a_gpu():
    lib = binding.load_library()
    assert lib.sja_destroy(None) == 0
    assert lib.sja_commit(None, None) == 1          # SJA_ERR_INVALID_ARG
    assert lib.sja_create(None, 0, None) == 1
    n = ctypes.c_uint64()
    assert lib.sja_scan_size(None, ctypes.byref(n)) == 1
    assert lib.sja_last_error(None) == b""


def test_workload_generators_are_deterministic_and_in_range():
    from paper_2509_19086_b200 import workloads as wl
    spec = wl.SPECS[0]
    a = wl.make_profiles(spec, threads=1)
    b = wl.make_profiles(spec, threads=4)
    for x, y in ((a.dur_ms, b.dur_ms), (a.mem_MiB, b.mem_MiB), (a.safe_bits, b.safe_bits),
                 (a.ready_ms, b.ready_ms)):
        assert np.array_equal(x, y)
    assert a.n_jobs == 64 and a.n_steps == 64 * 256
    assert a.dur_ms.min() >= 1 and a.dur_ms.max() <= 50
    assert a.mem_MiB.min() >= 1 and a.mem_MiB.max() <= 81920
    safe = wl.unpack_safe_bits(a.safe_bits, a.n_steps)
    assert safe[255::256].all()
    assert 0.05 < safe.mean() < 0.16
    g = wl.make_gaps(spec)
    assert g.shape == (16,) and set(np.unique(g["C_MiB"])) <= set(wl.CAPACITIES_MIB.tolist())
    assert g["T_ms"].min() >= 100 and g["T_ms"].max() <= 5000 and g["slice"].max() <= 6
    # ragged workload: lengths in range, block split independent of thread count
    sp3 = wl.scaled(wl.SPECS[3], n_jobs=300, zipf_max=3000)
    p1, p2 = wl.make_profiles(sp3, threads=1), wl.make_profiles(sp3, threads=3)
    assert np.array_equal(p1.mem_MiB, p2.mem_MiB) and np.array_equal(p1.safe_bits, p2.safe_bits)
    lens = np.diff(p1.off)
    assert lens.min() >= 16 and lens.max() <= 3000
    assert set(np.unique(p1.prio)) <= {0, 1, 2}
    # streaming workload: gap starts move with the round
    sp4 = wl.SPECS[4]
    g5 = wl.make_gaps(sp4, 5, n_gaps=64)
    assert g5["start_ms"].min() >= 5000 and g5["start_ms"].max() <= 7000
