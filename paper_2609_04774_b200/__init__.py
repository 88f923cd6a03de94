"""libcpattn: cache-aware causal prefill attention under zigzag context parallelism, for sm_100a.

The package holds the CUDA sources of the C-ABI library (``csrc/``), a thin ``ctypes`` binding
with the same names as the C entry points (``binding``), the build step (``build``) and the seeded
synthetic input generators (``workloads``).  Importing the package does not load the shared
library; the first call into ``binding`` does, and raises if the library has not been built.
"""
__all__ = ["binding", "build", "workloads"]
