"""B200-native IDKM hot path: soft k-means fixed point, soft quantiser, implicit / JFB backward.

``paper_2312_07759_b200.binding`` is the thin ctypes layer over the C-ABI library (it raises at
import if the library is missing); ``paper_2312_07759_b200.workloads`` holds the seeded inputs.
"""
__all__ = ["binding", "workloads", "build"]
