"""ShotKV hot path for NVIDIA B200: thin Python binding over the C-ABI library.

`binding` mirrors `include/shotkv.h` one to one (marshalling only); `workloads`
draws the seeded synthetic inputs; `build` compiles the CUDA library in-tree.
"""
from . import binding, workloads  # noqa: F401
from .binding import *  # noqa: F401,F403
from .binding import Context, Dims, Policy, DecodeState, ShotKVError, make_dims, make_policy  # noqa: F401
