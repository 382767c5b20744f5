"""B200-native MoSKA decode-attention hot path: CUDA kernels behind a C ABI, plus a thin binding.

`workloads` (seeded synthetic inputs) imports without the CUDA library; `binding` loads
`csrc/libmoska.so` and fails loudly if it is missing.
"""

__all__ = ["workloads", "binding", "build"]
