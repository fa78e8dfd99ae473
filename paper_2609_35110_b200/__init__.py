"""B200-native 3D-RoPE joint self-attention for video DiT blocks.

``workloads`` (seeded synthetic inputs) imports without a GPU; the CUDA path is
reached through ``paper_2609_35110_b200.binding``, which loads the C-ABI
library and raises if it has not been built.
"""
__all__ = ["workloads", "binding", "build"]
