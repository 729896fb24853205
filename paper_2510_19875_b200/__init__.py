"""B200-native Stream: hierarchical sparse-mask estimation and block-sparse attention.

``paper_2510_19875_b200.stream`` binds the C-ABI CUDA library; ``workloads`` makes seeded inputs.
Importing the package does not load the library; the first call into ``stream`` does, and fails
loudly if it has not been built.
"""
__all__ = ["stream", "workloads"]
