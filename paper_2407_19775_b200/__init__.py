"""B200-native dynamic blockwise 8-bit quantization of shard-boundary hidden states.

``workloads`` (seeded input generators) imports without the CUDA library; the binding
loads ``libbq.so`` on first use and raises if it has not been built.
"""
__all__ = ["workloads"]
