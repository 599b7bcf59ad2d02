"""B200-native SVD-Cache hot path: calibration (Gram + top-k eigenvectors), the fused
full step (project + residual + EMA) and the fused cached step (forecast + reconstruct),
as hand-written CUDA for sm_100a behind a C ABI.

``streams`` holds the seeded synthetic input generators; ``binding`` is the thin ctypes
layer over ``libsvdcache.so`` (argument marshalling only).  Importing the package does
not load the CUDA library; ``binding.lib()`` does, and raises if it is missing.
"""
__all__ = ["streams", "binding"]
