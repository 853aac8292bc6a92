"""B200-native (sm_100a) decode attention for Grouped Value Attention.

`binding` mirrors the C ABI of include/gva.h one to one; `workloads` draws the seeded synthetic
inputs; `harness` moves a generated case into device memory.  The compute lives in libgva.so
(hand-written CUDA); nothing here falls back to the CPU.
"""
from . import binding, workloads  # noqa: F401

__all__ = ["binding", "workloads"]
