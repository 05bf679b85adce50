"""B200-native SegLinear + DualScale W8A8 quantized linear layer (SegQuant hot path).

The product is the C-ABI shared library built from ``csrc/`` (hand-written CUDA
for sm_100a).  ``binding`` is the thin ctypes layer over it; ``workloads`` only
draws seeded synthetic inputs.  Importing the package does not load the library;
the first call through ``binding`` does, and fails loudly if it is missing.
"""
__all__ = ["binding", "workloads", "build"]
