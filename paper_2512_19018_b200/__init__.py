"""peak_gemm: B200-native dense GEMM (C = alpha*op(A)*op(B) + beta*C) behind a small C ABI.

`paper_2512_19018_b200.binding` holds the ctypes binding to the CUDA library;
`paper_2512_19018_b200.workloads` the seeded synthetic inputs.  Nothing is
loaded at import time, so the package imports on a machine without a GPU.
"""
__all__ = ["binding", "workloads", "build"]
