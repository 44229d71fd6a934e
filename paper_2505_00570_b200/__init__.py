"""FreqKV iterative KV-cache compression for B200 (sm_100a).

The product is the C-ABI library built from ``csrc/`` (declared in ``include/freqkv.h``);
``binding`` wraps it with the same names for Python callers, ``synth`` generates seeded
synthetic caches.  Importing the package does not load the library; the first call into
``binding`` does, and raises if the library has not been built.
"""

__all__ = ["binding", "synth"]
