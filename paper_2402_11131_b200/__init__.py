"""B200-native hot path of Speculative Streaming: multi-stream tree attention, greedy tree
verification and KV-cache compaction, as a C-ABI CUDA library with a thin ctypes binding.

``workloads`` (numpy only) draws the seeded synthetic inputs; ``api`` is the binding.  The CUDA
library is required: there is no CPU or PyTorch fallback, and ``api`` raises if it cannot load it.
"""
__all__ = ["workloads", "api", "build"]
