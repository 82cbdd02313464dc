"""KVSwap decode hot path for NVIDIA B200: CUDA kernels behind a C ABI (include/kvswap.h).

``binding`` mirrors the C entry points; ``workloads`` draws the seeded synthetic inputs;
``runtime`` holds marshalling helpers; ``build`` compiles libkvswap.so in-tree.
"""
__all__ = ["binding", "workloads", "runtime", "build"]
