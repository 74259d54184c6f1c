"""SIDCo gradient sparsifier for B200 (sm_100a): CUDA kernels behind a C ABI,
plus a thin ctypes binding.  Importing the package does not load the shared
library; the first call into :mod:`paper_2101_10761_b200.binding` does, and it
raises if the library has not been built."""

__all__ = ["binding", "workloads"]
