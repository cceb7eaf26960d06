"""B200-native KDA (Kimi Delta Attention) hot path: chunkwise prefill and recurrent decode.

The product is the CUDA library behind the C ABI declared in ``include/kda.h``; this package holds
its sources (``csrc/``), the build step and a thin ctypes binding with the same entry-point names
(``paper_2510_26692_b200.api``).  ``inputs`` draws the seeded synthetic workloads.
"""
