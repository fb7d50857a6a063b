"""B200-native multi-adapter LoRA forward: y = y_base + s_i * (x . A_i) . B_i.

The CUDA library is loaded lazily by :mod:`paper_2602_24044_b200.binding`;
:mod:`paper_2602_24044_b200.workloads` (seeded synthetic inputs) has no
dependency on it.
"""
__all__ = ["workloads", "binding", "build"]
