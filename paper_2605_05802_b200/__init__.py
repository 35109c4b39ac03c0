"""B200-native Selective Rollout gate: C-ABI CUDA library plus a thin binding.

``binding`` mirrors include/sr_gate.h one to one; ``workloads`` draws the seeded
synthetic inputs; ``build`` compiles the library in-tree for sm_100a.
"""
from .binding import *  # noqa: F401,F403
from .binding import load, SrError, shard_groups  # noqa: F401
