"""B200-native semantic draft pool (Oilbird retrieval hot path).

``paper_2608_03839_b200.binding`` is the thin ctypes layer over the C-ABI library built
from ``csrc/``; ``paper_2608_03839_b200.workloads`` draws the seeded synthetic inputs.
Nothing is imported eagerly so that CPU-only tools can use the workload generators
without the CUDA library being present.
"""
__all__ = ["binding", "workloads", "build"]
