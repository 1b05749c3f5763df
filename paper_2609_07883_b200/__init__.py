"""B200-native mixed prefill-chunk + decode attention iteration with the SLOWeave chunk controller.

Modules:

* ``build``      compiles ``csrc/`` into ``libsloweave.so`` with nvcc for sm_100a (``build_sanitized`` for the host sanitizers);
* ``binding``    a ctypes binding of the C-ABI declared in ``include/sw.h`` (argument marshalling only);
* ``workloads``  seeded synthetic input generators (numpy; no arithmetic of the method);
* ``profiler``   orchestration of ``sw_cost_probe``: cost tables for the controller and cost surfaces of the workloads;
* ``clocks``     SM clock / power / throttle record of a timed window (``nvidia-smi``, read only);
* ``serving``    the iteration-level serving loop (controller + executor + telemetry) over a request trace;
* ``simulate``   the paper's simulator study on the CPU (analytic cost model);
* ``sharding``   one iteration sharded by KV heads over several GPUs (no collective on the data path).

Importing the package itself loads nothing; ``binding`` raises if the shared library is missing (there is no fallback).
"""

__all__ = ["build", "binding", "workloads", "profiler", "clocks", "serving", "simulate", "sharding"]
