"""B200-native hot path of Tensor Homomorphic Compression (THC, arxiv 2302.08545).

``thc``        binding of the C-ABI library (prepare / compress / aggregate / decompress)
``workloads``  seeded synthetic gradients and parameter sets (shared with the tests' oracle)
``tables``     offline lookup-table solver (Section 5.2 / Appendix B), host only
``_build``     in-tree nvcc build of libthc.so for sm_100a
"""
__all__ = ["thc", "workloads", "tables"]
