"""B200-native MI hook: CUDA kernels behind a C ABI (include/mix.h) plus a thin binding."""
from .binding import *          # noqa: F401,F403
from .binding import Mix, MixError, load_library, set_pdl_mask  # noqa: F401
