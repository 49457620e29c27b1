"""B200-native double-sampled low-precision SGD for linear models (arxiv 1611.05402).

The work happens in hand-written CUDA kernels behind a C-ABI shared library; `binding` marshals
torch device tensors into those calls and `synth` draws the seeded synthetic workloads.
"""
__all__ = ["binding", "synth"]
