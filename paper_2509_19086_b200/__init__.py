"""B200-native SJA advertise / signal / select / commit round.

``workloads``  seeded synthetic inputs (no method arithmetic)
``binding``    thin ctypes binding of the C-ABI CUDA library ``libsja.so`` (see include/sja.h)
``build``      in-tree nvcc build of that library

There is no CPU fallback: using ``binding`` without the built library, or without a CUDA
device, raises.
"""
