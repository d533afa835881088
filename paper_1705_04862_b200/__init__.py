"""B200-native PAAC (parallel advantage actor-critic) hot path: a C-ABI CUDA library
(`libpaac_b200.so`, declared in include/paac.h) and this thin binding."""
from .binding import (ARCH_NATURE, ARCH_NIPS, BF16, FP32, Paac, PaacError, default_hparams, lib,  # noqa: F401
                      workspace_bytes)
from .configs import CONFIGS  # noqa: F401
