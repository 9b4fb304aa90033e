"""ConEF (contractive error feedback) step for B200: CUDA library + thin binding.

``workloads`` holds the synthetic parameter lists and seeded gradient
generators; ``binding`` loads the C-ABI library ``libconef.so`` (it raises if
the library is missing: there is no CPU fallback).  Nothing is imported
eagerly, so that the generators can be used without the CUDA library.
"""
__all__ = ["workloads", "binding"]
