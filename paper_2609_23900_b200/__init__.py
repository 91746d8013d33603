"""B200-native verifier hot path of LumoTree (path-parallel speculative verification of Gated DeltaNet
layers over a candidate tree, and the attention half of the same cycle).

``binding`` is the thin ctypes layer over the C-ABI CUDA library (``liblumo_gdn.so``, built by ``build.py``);
it raises if that library is missing: there is no CPU fallback.
"""
