"""B200-native ADMM-Q layer-wise quantization solver (CUDA for sm_100a behind a C ABI).

`binding` holds the ctypes marshalling over the shared library; `workloads` holds
the seeded synthetic input generators (no solver arithmetic).  Importing the
package does not load the shared library; the first solver call does, and it
raises if the library is missing.
"""
__all__ = ["binding", "workloads"]
