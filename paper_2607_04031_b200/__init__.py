"""B200-native tile-major GEMM hot path (relayout, tcgen05 GEMM, read-amplification count).

Importing the package is cheap and loads no native code; the C-ABI library is
loaded by ``paper_2607_04031_b200.binding`` on first use and every call fails
loudly when it is missing.  ``paper_2607_04031_b200.inputs`` (seeded synthetic
inputs) is self-contained.
"""
__all__ = ["binding", "inputs", "shard"]
