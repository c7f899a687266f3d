"""B200-native MLA decode over a paged latent KV cache (the attention hot path
under SPLASH's TP/DOP, DP-attention and CP layouts).

The CUDA library is loaded lazily by :mod:`paper_2609_37626_b200.binding`;
importing this package (e.g. for the seeded input generators in
:mod:`paper_2609_37626_b200.workloads`) does not need a GPU.
"""

__all__ = ["binding", "workloads", "build"]
