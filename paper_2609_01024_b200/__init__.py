"""Path-composed MoE FFN layer (PCoMoE) for NVIDIA B200: a C-ABI CUDA library
(``libpcomoe.so``, declared in ``include/pcomoe.h``) and a thin ctypes binding.

``workloads`` (seeded synthetic inputs) imports without the CUDA library;
everything in ``binding`` raises if the library is missing or cannot be loaded.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding", "build"]
