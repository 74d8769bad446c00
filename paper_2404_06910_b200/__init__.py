"""B200-native hot path of superposition prompting (arXiv 2404.06910).

Thin Python front-end of the C-ABI library ``libsp_b200.so`` (see ``include/sp.h``).
Importing this package loads the CUDA library; it raises if the library has not been
built.  There is no CPU or PyTorch fallback.
"""
from .binding import *  # noqa: F401,F403
from .binding import DeviceLayout, SpError, lib, EXPORTS, LIB_PATH, dtype_code  # noqa: F401
