"""B200-native graded KV-cache decode attention (Geodesia-KV hot path).

``binding`` wraps the C ABI of libgkv.so (CUDA, sm_100a); ``workloads`` draws the seeded
synthetic inputs; ``build`` compiles the library in tree.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding", "build"]
