"""B200 (sm_100a) decode hot path of Dynamic Thinking-Token Selection: fused GQA decode attention
+ importance accumulation over a budget-limited KV cache, and budgeted eviction with in-place
compaction.  The work is done by libdynts.so (CUDA); this package is its thin binding."""
from .binding import *  # noqa: F401,F403
from .binding import Cache, DyntsError, lib, LIB_PATH  # noqa: F401
