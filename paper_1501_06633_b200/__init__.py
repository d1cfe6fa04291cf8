"""B200-native FPROP direct convolution (maxDNN's hot path)."""
from . import workloads  # noqa: F401
