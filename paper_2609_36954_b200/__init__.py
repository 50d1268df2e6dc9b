"""B200-native collectives executor: C-ABI library (libpurlin.so) plus a thin ctypes binding.

``binding`` mirrors the C entry points one to one; ``inputs`` holds the seeded synthetic
input generators.  The datapath runs only in the CUDA library; there is no CPU fallback.
"""
from . import binding, inputs  # noqa: F401

__all__ = ["binding", "inputs"]
