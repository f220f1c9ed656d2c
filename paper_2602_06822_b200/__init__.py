"""POP (partition-guided online pruning) hot path for NVIDIA B200 (sm_100a).

``paper_2602_06822_b200.pop``        thin ctypes binding over the C-ABI library (libpop.so)
``paper_2602_06822_b200.workloads``  seeded synthetic inputs (no method arithmetic)

Importing the package does not load the CUDA library; ``pop.lib()`` does, and
raises if it has not been built.
"""
__version__ = "0.1.0"
