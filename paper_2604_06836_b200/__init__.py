"""B200-native mixed-bit quantized AdamW step (the STQuant optimizer hot path).

``stq`` is the thin binding over the C-ABI library built from ``csrc/``; ``workloads`` holds the
seeded synthetic parameter sets.  Importing the package does not load the CUDA library; the first
call into ``stq`` does, and fails loudly if it has not been built.
"""
__all__ = ["stq", "workloads"]
