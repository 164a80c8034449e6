"""B200-native decode attention over a segment KV cache (beam-index selection fused).

``segkv``      ctypes binding of the C-ABI library (CUDA kernels for sm_100a)
``workloads``  seeded synthetic inputs of the evaluation shapes
``build``      compiles ``libsegkv.so`` in-tree with nvcc
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "segkv", "build"]
