"""B200 (sm_100a) quantized-linear kernels for DVD-Quant's inference hot path.

``binding`` exposes the C ABI of ``include/dvdq.h`` with the same names; ``build``
compiles the CUDA library in-tree; ``workloads`` holds the seeded synthetic inputs.
"""
from . import binding, build, dist, workloads  # noqa: F401

__all__ = ["binding", "build", "dist", "workloads"]
