"""APMSqueeze compressed-step hot path for NVIDIA B200: CUDA library + thin binding."""
from . import binding, workloads  # noqa: F401
from .binding import Context  # noqa: F401
