"""B200-native zero-value compression (ZVC) of activation maps and the
compressed offload / prefetch copy built on it (the cDMA method).

``binding``   -- ctypes front end of the C-ABI CUDA library (``libcdma.so``).
``workloads`` -- seeded synthetic activation maps (inputs only).

The codec exists only as CUDA kernels for sm_100a; there is no CPU path.
"""
from . import binding, workloads  # noqa: F401

__all__ = ["binding", "workloads"]
