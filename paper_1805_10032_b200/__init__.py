"""Zeno aggregation step (stochastic descendant score, ranking, trimmed mean)
as hand-written CUDA for sm_100a behind a small C ABI.

`paper_1805_10032_b200.zeno` is the ctypes binding of the shared library built
from `csrc/`; `paper_1805_10032_b200.synthetic` builds seeded inputs.
"""
__all__ = ["zeno", "synthetic"]
