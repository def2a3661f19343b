"""B200-native exact integer matrix products on FP4 tensor cores (Adaptive Weight Encoding).

The CUDA library is loaded lazily by `paper_2609_24519_b200.binding`; importing the
package itself needs no GPU.
"""
__all__ = ["binding", "workloads"]
