"""B200-native Collage bf16 MCF AdamW step: C-ABI CUDA library plus a thin Python binding.

``binding`` holds the ctypes front end of the CUDA library (loaded on first use, fails
loudly if the library was not built); ``workloads`` holds the seeded synthetic inputs.
"""
__all__ = ["binding", "workloads"]
