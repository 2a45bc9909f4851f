"""B200-native data-parallel hot path of Slow Momentum (SlowMo, arXiv 1910.00643).

`binding` wraps the C-ABI library libslowmo.so (include/slowmo.h); `workloads` describes the
seeded synthetic inputs; `build` compiles the CUDA sources for sm_100a. The library is loaded
on first use and there is no CPU fallback.
"""
from . import workloads  # noqa: F401
from .binding import SlowMo, SlowMoError, lib  # noqa: F401
