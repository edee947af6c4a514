"""Focus-dLLM per-step sparse-attention path for NVIDIA B200: ctypes binding of libfocus.so plus the
seeded synthetic workloads used by tests and benchmarks."""
from . import workloads  # noqa: F401
from .binding import *  # noqa: F401,F403
from .binding import Context, FocusError, focus_shape, load_library, make_shape  # noqa: F401
