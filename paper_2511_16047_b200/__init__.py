"""AMS-KV hot path for NVIDIA B200: segmented per-layer KV cache, scale-adaptive attention
and inter-scale key similarity, as CUDA kernels behind a small C ABI (include/amskv.h).

`binding` mirrors the C ABI one to one; `synth` makes seeded synthetic workloads.
Importing this package loads libamskv.so and fails if it has not been built.
"""
from . import binding, synth  # noqa: F401
from .binding import *  # noqa: F401,F403
