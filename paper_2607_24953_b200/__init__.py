"""fp4q: transposition-invariant 2D-block FP4 quantization and block-scaled GEMMs for B200 (sm_100a).

The product is the C-ABI library ``libfp4q.so`` (declared in ``include/fp4q.h``); ``binding`` is its
thin Python face and ``workloads`` the seeded synthetic input generators.
"""
__all__ = ["binding", "workloads", "build", "autograd"]
