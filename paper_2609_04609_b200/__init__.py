"""B200-native exponent-reuse codec (CIERA hot path): C-ABI library + thin binding.

``paper_2609_04609_b200.ciera``      ctypes binding of ``libciera.so`` (loads the CUDA library;
                                     raises if it has not been built)
``paper_2609_04609_b200.workloads``  seeded synthetic inputs (no codec arithmetic)
"""
__all__ = ["ciera", "workloads"]
