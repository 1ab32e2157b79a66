"""B200-native tree-verification step for Clover-2-style speculative decoding.

``binding`` forwards to the C ABI of libclv.so (hand-written sm_100a kernels); ``step`` keeps the
device buffers of one verify step; ``workloads`` makes seeded synthetic inputs.  Nothing here
falls back to the CPU: without the built library every call raises.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads"]
