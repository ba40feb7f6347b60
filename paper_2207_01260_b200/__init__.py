"""B200 (sm_100a) task execution for channel-pruned CNNs: fused conv + bias + activation tasks at
arbitrary pruned channel counts and L1-norm filter selection, behind the C ABI of include/cprune.h.

``binding`` mirrors the C entry points one to one (argument marshalling only); ``pipeline`` strings
those calls together for a whole pruned network.  Nothing here computes on the CPU: without the
compiled library (``python -m paper_2207_01260_b200.build``) every call raises.
"""
from . import binding  # noqa: F401
from .binding import *  # noqa: F401,F403
