"""B200-native shared-attention (SAN) decode path.

The package holds three things and nothing else:

* ``synth``   -- seeded synthetic workloads (no attention arithmetic),
* ``build``   -- compiles ``csrc/`` into ``libsan_b200.so`` for sm_100a,
* ``binding`` -- a ctypes binding with the same names as ``include/san.h``.

Importing the package does not load the CUDA library; ``binding.lib()`` does,
and raises if the library has not been built.
"""

__all__ = ["synth", "build", "binding"]
