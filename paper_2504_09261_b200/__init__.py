"""B200 (sm_100a) library for the per-scale decoding step of head-aware KV-cache compression.

The product is the C-ABI shared library declared in include/hack.h; this package holds its CUDA
sources (csrc/), the build script and a ctypes binding with the same names as the C entry points.
"""
from .binding import (  # noqa: F401
    HACK_BF16, HACK_F32, HACK_OBS_CALLER, HACK_OBS_FULL, HACK_OBS_INIT, HACK_OBS_RECENT, HACK_OBS_UNIFORM, HACK_OK, HACK_OVERFLOW_COMPETE, HACK_OVERFLOW_KEEP_PROTECTED, RULE_FRACTION,
    RULE_RATIO, EXPORTS, HackCache, HackError, hack_classify_heads, hack_last_error, hack_score_noalloc, hack_split_budget,
)
