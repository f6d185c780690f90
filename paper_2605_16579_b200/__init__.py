"""ARL^2 hybrid attention layer for B200 (sm_100a): a C-ABI CUDA library plus this thin binding.

``paper_2605_16579_b200.arl2`` holds the ctypes binding of the library (argument
marshalling only); ``paper_2605_16579_b200.workload`` holds the seeded synthetic input
generators.  Importing the package itself loads nothing.
"""

__all__ = ["arl2", "workload"]
