"""B200-native GDN tree verify + commit (path-parallel speculative verification of
Gated DeltaNet layers over a candidate tree).

``workload`` holds the seeded synthetic inputs; ``binding`` is the thin ctypes layer over
the C-ABI CUDA library (``liblumo_gdn.so``, built by ``build.py``) and raises if that
library is missing: there is no CPU fallback.
"""
from . import workload  # noqa: F401

__all__ = ["workload"]
