"""B200-native (sm_100a) hybrid attention layer of NAtS-L: hand-written CUDA kernels behind a
C-ABI library (``include/natsl.h``) and a thin ctypes binding with the same names.

``inputs`` (seeded synthetic workloads) imports without the CUDA library; everything in
``binding`` needs the built library and fails loudly without it -- there is no CPU fallback.
"""
__all__ = ["inputs", "binding", "build"]
