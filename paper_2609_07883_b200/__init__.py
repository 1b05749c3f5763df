"""B200-native mixed prefill-chunk + decode attention iteration with the SLOWeave chunk controller.

The package holds three things only:

* ``workloads``  seeded synthetic input generators (numpy; no arithmetic of the method);
* ``build``      compiles ``csrc/`` into ``libsloweave.so`` with nvcc for sm_100a;
* ``binding``    a ctypes binding of the C-ABI declared in ``include/sw.h``.

Importing the package itself loads nothing; ``binding`` raises if the shared library is missing.
"""

__all__ = ["workloads", "build", "binding"]
