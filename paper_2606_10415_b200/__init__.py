"""B200-native FP16 causal / grouped-query attention forward and backward.

The product is a C-ABI CUDA library (``csrc/``, declared in ``include/lt_attn.h``);
``binding`` marshals torch device pointers into it and ``workloads`` draws the
seeded benchmark inputs.  Nothing here falls back to the CPU: importing
``binding`` raises if the compiled library is missing.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads"]
