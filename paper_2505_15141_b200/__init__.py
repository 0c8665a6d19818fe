"""B200-native batched speculative-decoding verification with bandit-chosen speculation length.

Submodules:
  binding    -- thin ctypes layer over the C-ABI library (loads the CUDA extension; raises if absent)
  workloads  -- seeded synthetic inputs (no verification arithmetic, no native code)
"""
__all__ = ["binding", "workloads"]
