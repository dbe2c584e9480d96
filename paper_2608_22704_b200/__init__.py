"""B200-native (sm_100a) decode hot path of the WnW KV cache behind a C ABI (include/wnw.h)."""
from .binding import *  # noqa: F401,F403
from .binding import lib, library_path, exported_symbols, status_string, WnwError  # noqa: F401
