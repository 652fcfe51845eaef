"""CPU checker for the quantized linear layer (test infrastructure, not a product path).

Thin ctypes/numpy marshalling around ``aq_oracle.cpp``; all arithmetic lives in the
C++ file. Only tests, the smoke check and the benchmark's CPU-baseline leg use it.
The CUDA library never does.
"""
from .binding import *  # noqa: F401,F403
