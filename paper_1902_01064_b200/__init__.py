"""Hop (heterogeneity-aware decentralized SGD, arXiv 1902.01064) hot path for one B200.

Sub-modules:
  inputs   seeded synthetic workloads (graphs, compute-time tables, SVM shards, p_0);
           holds none of the method's arithmetic and never touches the GPU.
  build    compiles csrc/ into libhop_b200.so with nvcc for sm_100a.
  hop      ctypes binding of the C ABI declared in include/hop.h.  Importing it
           loads the shared library and raises if it is missing: there is no
           CPU fallback for the product path.
"""

__all__ = ["inputs", "build", "hop"]
