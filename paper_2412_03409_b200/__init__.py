"""B200-native PrefixKV hot path: C-ABI CUDA library plus a thin Python binding.

``paper_2412_03409_b200.api`` loads the shared library and mirrors its entry
points; ``paper_2412_03409_b200.workloads`` holds the seeded input generators.
Importing this package alone loads no native code.
"""
__all__ = ["api", "workloads"]
