"""B200-native VIA-SD multi-tier verification step: CUDA kernels behind a C ABI, plus a thin binding."""
from . import binding  # noqa: F401
