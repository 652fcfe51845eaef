"""Agile-Quant's quantized linear layer for B200 (sm_100a): hand-written CUDA kernels behind
a C-ABI library (``include/agileq.h``) and a thin ctypes binding (``binding``).

Importing the package does not load the CUDA library; ``binding.load()`` does, and raises if
it has not been built (``python -m paper_2312_05693_b200.build``). There is no fallback path.
"""
from . import inputs  # noqa: F401

__all__ = ["inputs", "binding", "build"]
