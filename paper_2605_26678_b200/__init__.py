"""B200-native NestedKV compression hot path (anchors, scoring, budgets, selection, compaction).

The CUDA library is loaded lazily by :mod:`paper_2605_26678_b200.nkv`; importing the package
(for instance to reach the synthetic workload generator) does not need a GPU.
"""
__all__ = ["workloads"]
