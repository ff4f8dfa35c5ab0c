"""B200-native SpMM for moderately (~50 %) unstructured sparse fp16 weights in the paper's
three-layer format (Sparse-TC + Slot-Filling with PDD codes + Residual).

``from paper_2607_08786_b200 import tl3`` gives the Python binding of the C-ABI library
(``include/tl3.h``); it raises at first use if the CUDA library has not been built.
``workloads`` holds the seeded synthetic input generators and needs only numpy.
"""
__all__ = ["tl3", "workloads"]
