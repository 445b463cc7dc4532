"""B200-native fused multi-agent rollout + GAE (C-ABI CUDA library and its thin binding).

``workloads`` holds the seeded synthetic inputs; ``binding`` loads the CUDA
shared library lazily (and raises if it has not been built).
"""
from . import workloads  # noqa: F401

__all__ = ["workloads"]
