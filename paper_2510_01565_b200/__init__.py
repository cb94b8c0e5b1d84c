"""B200-native single-GPU DiT denoising step (packed mixed-resolution batch).

`workloads` draws seeded synthetic inputs; `binding` loads the C-ABI CUDA
library (libdit.so) and is imported lazily so that input generation works on
machines without a GPU.
"""
__all__ = ["workloads", "binding"]
