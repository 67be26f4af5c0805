"""B200-native ROBE-Z embedding lookup (arXiv 2108.02191): a C-ABI CUDA library
(``librobe.so``, declared in ``include/robe.h``) and this thin binding of it."""
from .binding import *  # noqa: F401,F403
from .binding import EXPORTS, LIB_PATH, RobeError  # noqa: F401
