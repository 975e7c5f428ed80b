"""hct: fused operator-chain execution on NVIDIA B200 through a C-ABI library (include/hct.h).

The Python layer only marshals arguments; every step of a chain runs in CUDA kernels that the
library generates and compiles for sm_100a.  There is no CPU or framework fallback.
"""
from .binding import *  # noqa: F401,F403
from .binding import HctError, lib  # noqa: F401
from .graph import FusedGraph  # noqa: F401
