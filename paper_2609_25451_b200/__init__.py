"""B200-native restore / digest / verify data path of a GPU Memory Service.

``gms``        ctypes binding of the C ABI (include/gms.h); the only compute path.
``workloads``  seeded synthetic layouts and random contents for tests and the benchmark.
``build``      compiles ``libgms.so`` in-tree with nvcc for sm_100a.
"""
from . import gms, workloads  # noqa: F401

__all__ = ["gms", "workloads"]
