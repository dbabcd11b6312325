"""libape for B200: APE (Adaptive Parallel Encoding) attention as hand-written sm_100a CUDA kernels.

``paper_2502_05431_b200.libape`` is the thin ctypes binding over the C-ABI library
(``include/ape.h``); ``paper_2502_05431_b200.workloads`` draws the seeded synthetic inputs.
"""
