"""B200-native (sm_100a) MoE-layer forward for SPICE-style offloaded decoding.

The product is the C-ABI library `libspice.so` (see include/spice.h); this package holds its
CUDA sources (`csrc/`), the build step (`build.py`), a thin ctypes binding with the same entry
point names (`binding.py`) and the seeded synthetic workload generator (`workloads.py`).
Importing the package loads nothing; the binding loads the library on first use and raises if
it is missing -- there is no CPU fallback.
"""

__all__ = ["binding", "build", "workloads"]
