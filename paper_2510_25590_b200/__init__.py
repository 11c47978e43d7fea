"""B200-native region-aware denoising step (RegionE hot path).

``synth`` holds the seeded input generators; ``binding`` is the thin ctypes
layer over the C-ABI library ``libregione.so`` built from ``csrc/``.  Nothing
is loaded at import time; the binding raises if the library is missing.
"""
