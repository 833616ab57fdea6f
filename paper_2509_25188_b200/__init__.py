"""Learn2PD decoding on B200: C-ABI CUDA library plus a thin Python binding.

`workloads` (seeded synthetic inputs, numpy only) can be imported without the
CUDA library; `binding` loads the shared library and fails loudly if it is missing.
"""
__all__ = ["workloads", "binding"]
