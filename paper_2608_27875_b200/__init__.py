"""B200-native (sm_100a) HyQuant prefill path: vertical-line selection,
per-block low-bit quantization and the fused hybrid-precision causal attention
forward, behind a C-ABI shared library (``include/hyq.h``).

``workloads`` (seeded synthetic inputs) imports without the CUDA library; the
binding in ``api`` raises as soon as it is used if the library is missing.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads"]
