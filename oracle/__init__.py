"""CPU oracle for the SJA round -- TEST INFRASTRUCTURE ONLY.

Only ``tests/``, ``__graft_entry__.smoke()`` and the CPU-baseline legs of ``bench.py``
may import this package.  It shares nothing with the CUDA path and does not import it.

Contents
--------
``sja_oracle.c``   the naive step-by-step walk (R1-R6 in its header), built with gcc
``brute.py``       exhaustive prefix enumeration in pure Python, for tiny inputs
``scan.py``        the per-job prefix quantities written out with numpy
``api.py``         ctypes wrapper around the compiled walk
``reauction.py``   the round repeated for gaps orphaned by multi-winners (built from the walk)
``fast_oracle.c``  a second, separately written oracle (dense prefix arrays + binary search), built with gcc;
``fast.py``        its ctypes wrapper
``trajectory.py``  full-size trajectories reduced to fingerprints (what tests/golden/ stores)
"""
from .api import (  # noqa: F401
    AWARD_DTYPE,
    GAP_DTYPE,
    NO_JOB,
    commit,
    commit_masked,
    num_threads,
    pair,
    select,
)
from .brute import brute_pair, brute_select  # noqa: F401
from .reauction import round_with_reauction  # noqa: F401
from .scan import boundary_table, dense_prefix  # noqa: F401


def build(force: bool = False) -> str:
    """Compile both C oracles (the walk and the prefix-array oracle) next to their sources; returns the walk's path."""
    from . import api, fast

    fast.build(force)
    return api.build(force)
