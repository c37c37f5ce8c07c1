"""B200-native first-layer cached attention (RoPECache + FACache of LaCache).

The compute lives in the CUDA library built from ``csrc/`` and is reached
through ``paper_2607_16339_b200.binding`` (a thin ctypes layer over the C ABI
declared in ``include/lacache.h``).  Importing the package does not load the
library; the first use of the binding does, and fails loudly if it is missing.
"""
__all__ = ["binding", "workloads"]
