"""Prob-sparse multi-head self-attention (arXiv 2106.09236, Sec. 3) for NVIDIA B200.

The product is the CUDA library behind ``include/psattn.h``; this package holds
its sources (``csrc/``), a thin ctypes binding with the same names
(``binding``) and the seeded input generators (``workloads``).  The library is
loaded on first use of the binding, not at import.
"""
__all__ = ["workloads", "binding"]
