"""Binarized Bi-GCN forward layer for NVIDIA B200 (sm_100a): hand-written CUDA kernels behind a
C ABI (``include/bigcn.h``) and a thin ctypes binding (``paper_2210_13149_b200.binding``)."""

__all__ = ["binding", "synth", "build"]
