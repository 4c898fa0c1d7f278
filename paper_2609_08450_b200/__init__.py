"""B200-native exact Top-K selection for ragged FP32 sparse-attention score rows.

The product is the C-ABI library built from ``csrc/`` (declared in
``include/hpctopk.h``); ``binding`` is a thin ctypes layer with the same names,
``workloads`` holds the seeded synthetic input recipes.
"""
__version__ = "0.1.0"
