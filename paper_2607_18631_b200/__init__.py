"""B200-native batched scoring of MoE parallel-plan candidates (hand-written CUDA behind a C ABI).

`binding` is a thin ctypes layer over libplanfront.so (built in-tree by `build`); there is no CPU path.
"""
from . import binding  # noqa: F401
from .binding import Plan, PlanfrontError, pf_topk_merge, pf_version  # noqa: F401
