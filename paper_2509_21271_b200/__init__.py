"""B200-native bucketized speculative AdamW (SuperOffload's optimizer hot path).

The CUDA library is reached through :mod:`paper_2509_21271_b200.binding`
(loaded on first use; it raises if the compiled library is missing).
"""
__all__ = ["binding", "workloads", "build"]
