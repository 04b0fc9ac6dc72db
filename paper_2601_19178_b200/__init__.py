"""CollectiveKV decode-stage hot path for NVIDIA B200: a C-ABI CUDA library (libckv.so,
declared in include/ckv.h) and this thin Python binding.  PyTorch is used by callers only
for device memory and streams."""
from .binding import *  # noqa: F401,F403
from .binding import CkvError, EXPORTS, LIB_PATH, lib  # noqa: F401
from .session import CollectiveKV  # noqa: F401
