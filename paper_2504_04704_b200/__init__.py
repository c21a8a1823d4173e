"""LagKV KV-cache compression pass for NVIDIA B200 (sm_100a).

``paper_2504_04704_b200.binding`` wraps the C-ABI CUDA library; ``synth`` holds the
seeded input generators.  Importing the package loads nothing native: the shared
library is opened on the first call into ``binding`` and a missing library is an error.
"""
__all__ = ["binding", "synth", "shard"]
