"""B200-native forward pass of the Hybrid Gated Flow (HGF) dual-stream linear layer.

The compute lives in a C-ABI CUDA library (csrc/, built to libhgf_b200.so); `hgf` is the thin
ctypes binding with the same entry-point names.  `inputs` holds the seeded synthetic workloads.
Importing this package loads nothing; the CUDA library is loaded on first use of `hgf`.
"""
__all__ = ["hgf", "inputs", "build"]
