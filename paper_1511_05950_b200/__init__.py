"""n-softsync parameter-server update (arXiv 1511.05950) as sm_100a CUDA kernels behind a C ABI.

`binding` loads libsoftsync_ps.so and mirrors its entry points; build it first with
`python -m paper_1511_05950_b200.build`.
"""
from .binding import *  # noqa: F401,F403
from .binding import ParameterServer, SoftsyncError, lib  # noqa: F401
