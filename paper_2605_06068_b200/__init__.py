"""B200-native batched decode attention over a paged KV cache.

``kv_append`` -> ``paged_decode_attention`` -> ``paged_decode_reduce`` are
hand-written sm_100a CUDA kernels behind a C ABI (``include/pda.h``); this
package is the thin ctypes binding plus the seeded input generators.
Importing the package never loads the shared library; the first call does and
fails loudly if it has not been built.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads"]
