"""QA-LoRA linear layer (arXiv 2309.14717) as hand-written sm_100a CUDA kernels
behind a C-ABI library; this package holds the kernels' sources, the build
step and a thin ctypes binding."""

__all__ = ["binding", "synthetic", "build"]
