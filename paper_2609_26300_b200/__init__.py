"""CompKV decode hot path for B200 (sm_100a): C-ABI CUDA library plus a thin binding.

Importing the package does not load the CUDA library; `paper_2609_26300_b200.binding`
loads it on first use and raises if it has not been built.
"""
__all__ = ["synth", "binding", "build"]
