"""B200-native hot path of Tensor Homomorphic Compression (THC, arxiv 2302.08545).

``thc``        binding of the C-ABI library (prepare / compress / aggregate / decompress)
``workloads``  seeded synthetic gradients and parameter sets (shared with the tests' oracle)
``_build``     in-tree nvcc build of libthc.so for sm_100a
"""
__all__ = ["thc", "workloads"]
