"""B200-native operator layer for Relay programs: the fused primitive-operator groups
(dense / conv2d anchors with bias + activation epilogues, broadcast-elementwise and reduce
groups, their gradient groups, and an LSTM sequence) as hand-written sm_100a kernels behind a
C ABI (include/relay_b200.h).  `binding` is the ctypes front end; `build` compiles the library.
"""
from . import binding  # noqa: F401  (the library itself is loaded on first use and must exist)

__all__ = ["binding"]
