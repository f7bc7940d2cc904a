"""GradiVeQ's data-parallel hot path as hand-written sm_100a CUDA kernels behind a C ABI.

``paper_1811_03617_b200.gvq`` is the thin binding of the shared library
(``libgvq.so``, built by ``paper_1811_03617_b200.build``); ``workloads`` draws
the seeded synthetic inputs.  Importing the package loads nothing; the first
use of the binding loads the library and fails loudly if it is missing.
"""
__all__ = ["gvq", "workloads", "build", "replicas"]
