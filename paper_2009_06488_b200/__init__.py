"""B200-native 4-bit quantized GEMM and GEMM-based convolution (sm_100a).

The compute path lives in the CUDA library built from ``csrc/`` and is reached
through the C ABI declared in ``include/q4.h``; :mod:`.binding` is the thin ctypes
layer over it (argument marshalling only).  :mod:`.workloads` draws the seeded
synthetic inputs.  Nothing in this package computes on the CPU: importing
:mod:`.binding` without the built library raises.
"""
__all__ = ["binding", "workloads", "build"]
