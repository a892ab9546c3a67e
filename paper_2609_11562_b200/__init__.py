"""B200-native fused GEMM-ReduceScatter (Entwine), one-rank emulation.

`paper_2609_11562_b200.entwine` is the ctypes binding over the C-ABI library (it raises if
the CUDA library has not been built); `paper_2609_11562_b200.inputs` draws the seeded
synthetic operands.  Nothing is imported eagerly here so that the input generators can be
used without the compiled library.
"""
__all__ = ["entwine", "inputs", "build"]
