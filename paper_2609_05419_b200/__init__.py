"""2M complex matrix multiplication (2M multiplication + Ozaki-II) for NVIDIA B200 (sm_100a).

The product is the C-ABI library built from ``csrc/`` (declared in ``include/gemm2m.h``);
``binding`` is a thin ctypes layer with the same entry-point names, ``inputs`` holds the seeded
synthetic input generators.  There is no CPU fallback: using ``binding`` without the built CUDA
library raises.
"""
__all__ = ["binding", "inputs", "build"]
