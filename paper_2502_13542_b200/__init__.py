"""B200-native ActQKV per-window retrieval path (arXiv 2502.13542).

`paper_2502_13542_b200.binding` is the thin Python layer over the C-ABI CUDA
library; `paper_2502_13542_b200.workloads` draws the seeded synthetic inputs.
Nothing here computes any step of the method on the CPU.
"""
__all__ = ["workloads"]
