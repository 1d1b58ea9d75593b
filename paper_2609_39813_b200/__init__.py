"""Backward-state-policy operators and their per-use Monte-Carlo check on NVIDIA B200.

The product is the C-ABI library built from csrc/ (declared in include/bsp.h); `binding`
exposes the same entry points to Python, `workloads` draws the seeded synthetic inputs.
Nothing here computes on the CPU: without the built library and a CUDA device every entry
point raises.
"""
from . import workloads  # noqa: F401  (numpy only)

__all__ = ["binding", "workloads", "build"]
