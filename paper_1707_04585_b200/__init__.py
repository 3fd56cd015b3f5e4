"""B200-native reversible residual network hot path (CUDA kernels behind a C ABI)."""
from . import synthetic  # noqa: F401
