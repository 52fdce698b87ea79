"""B200 (sm_100a) GPTAQ per-layer solve: ctypes binding over libgptaq.so."""
from .binding import *  # noqa: F401,F403
from .binding import LayerState, GptaqError, load_library, LIB_PATH, SIGNATURES  # noqa: F401
