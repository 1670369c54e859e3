"""B200-native ternary pointwise convolution (the hot path of PROM).

The package is a thin binding over a C-ABI CUDA library (``csrc/``): every
step of the path runs in hand-written sm_100a kernels.  ``synth`` holds the
seeded input generators and workload tables; ``binding`` loads the library.
Nothing is loaded at import time.
"""
__all__ = ["synth", "binding", "build"]
