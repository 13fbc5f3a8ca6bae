"""MixKVQ decode hot path for B200: C-ABI CUDA library plus a thin ctypes binding.

``binding`` loads the shared library (and fails loudly if it is missing); ``workloads`` generates the
seeded synthetic inputs and holds none of the method's arithmetic.  Nothing is imported eagerly so
that ``workloads`` can be used on a machine without the library.
"""

__all__ = ["binding", "workloads"]
