"""B200-native sparse drafter linears (SD^2 decode hot path).

The package holds three things and nothing else:

* ``synth``   -- seeded synthetic inputs (weights, masks, activations).  It holds
  none of the method's arithmetic and is the only module that both the CPU
  oracle's tests and the CUDA path's tests draw inputs from.
* ``binding`` -- a thin ctypes layer over ``libsd2.so`` (argument marshalling
  only; every step of the path runs in the CUDA kernels behind the C ABI).
* ``build``   -- compiles ``csrc/`` into ``libsd2.so`` for sm_100a, in-tree.

Importing the package is cheap and has no side effects; the shared library is
loaded on first use of ``binding`` and a missing library is a hard error
(there is no CPU fallback).
"""

__all__ = ["synth", "binding", "build"]
