"""B200-native (sm_100a) template-recovery factorization for TSID matrix completion.

The product is the C-ABI library built from ``csrc/`` (declared in ``include/tsid.h``);
``binding`` is the thin ctypes layer over it and ``workloads`` the seeded input
generators.  Importing the package is cheap; the CUDA library is loaded on first use
and a missing library raises (there is no CPU fallback).
"""

__all__ = ["binding", "workloads", "build"]
