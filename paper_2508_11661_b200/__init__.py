"""SamKV hot path for NVIDIA B200 (sm_100a): scoring, per-context top-k, compaction,
recompute write-back and GQA attention over a multiple-context KV cache, as a C-ABI
CUDA library (`libsamkv.so`) plus this thin Python binding.

Importing the package does not load the CUDA library; `binding.lib()` does, and raises
if it has not been built (there is no CPU fallback).
"""
__all__ = ["binding", "synth", "build"]
