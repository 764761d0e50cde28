"""B200-native CSER / M-CSER optimizer step (arXiv 2007.13221) behind a C ABI.

``paper_2007_13221_b200.binding`` wraps ``libcser.so`` (hand-written CUDA for
sm_100a); ``synth`` holds the seeded synthetic workloads; ``shard`` the
column-slab partition used when several GPUs each own part of the vector.
Importing the package does not load the CUDA library; the first use of the
binding does, and raises if the library has not been built.
"""
__all__ = ["binding", "synth", "shard"]
