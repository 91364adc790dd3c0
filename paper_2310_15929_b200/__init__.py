"""E-Sparse hot path for NVIDIA B200: 2:4 pruning metric + shuffle + compression and the sparse GEMM.

`binding` wraps the C ABI declared in include/esparse.h (built from csrc/ by `build`); `inputs` holds the
seeded synthetic workloads.  Importing `binding` requires the compiled library: there is no fallback.
"""
