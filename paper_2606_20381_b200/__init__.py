"""B200-native UFP4 hot path: fused RHT + block-scaled uniform 4-bit quantizer and the 4-bit block-scaled training
GEMMs (fwd_y, bwd_dx, bwd_dw, plus the MoE-grouped variant), as a C-ABI CUDA library with a thin ctypes binding.

`inputs` draws the synthetic workloads; `binding` marshals arguments to libufp4.so (every step of the path runs in
the library's CUDA kernels; there is no CPU fallback and a missing library raises on first use).
"""
__all__ = ["inputs", "binding", "recipe"]
