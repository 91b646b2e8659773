"""B200-native fused AllGather+GEMM / GEMM+ReduceScatter (Compass hot path).

Importing the package does not load the native library; the first call into
``paper_2609_10549_b200.api`` does, and fails loudly if it was not built
(``python -m paper_2609_10549_b200.build``).  There is no CPU fallback.
"""
__all__ = ["workloads"]
