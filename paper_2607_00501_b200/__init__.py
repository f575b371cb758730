"""Block-quantised (Q4/Q8) dequantise-and-multiply kernels for B200 (sm_100a).

``paper_2607_00501_b200.qmm`` is the thin ctypes binding of ``libqmm.so`` (the
C-ABI declared in ``include/qmm.h``); ``paper_2607_00501_b200.synth`` makes the
seeded synthetic inputs.  Nothing here falls back to a CPU implementation: if
the CUDA library is missing, the first call raises.
"""
__all__ = ["qmm", "synth"]
