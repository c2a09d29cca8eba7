"""B200-native KV substrate hot path (prefix match, KV offload/restore, D2D staging).

The CUDA library is loaded lazily by :mod:`paper_2607_17181_b200.binding`; importing
the package (for example to reach :mod:`workloads`) does not need a GPU.
"""
__all__ = ["binding", "workloads", "replay", "replicas", "bench_configs"]
