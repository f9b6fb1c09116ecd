"""B200-native FAST-AR attention step: TempCache update, AnnSA and AnnCA as hand-written
sm_100a CUDA kernels behind a C-ABI library (see include/fastar.h).

`paper_2602_01801_b200.fastar` is the thin Python binding (ctypes; torch only for device
memory and streams); `paper_2602_01801_b200.synth` draws the seeded synthetic workloads.
Nothing is imported eagerly so that the workload generator works without the CUDA library.
"""
__all__ = ["fastar", "synth"]
