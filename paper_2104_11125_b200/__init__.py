"""B200-native CLT-k compression step of ScaleCom (Algorithm 1): C-ABI CUDA library + thin binding."""
from .binding import Context, ScaleComError, lib, strerror  # noqa: F401
from . import binding, workloads  # noqa: F401
