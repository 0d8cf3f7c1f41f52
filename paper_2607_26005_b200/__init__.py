"""B200-native batched egocentric rasterizer (class u8 + depth f16 per agent camera).

The work is done by libpictura.so (hand-written CUDA for sm_100a, C ABI in include/pictura.h);
this package is the thin Python binding used by the tests and the benchmark.
"""
from . import build
from .binding import (Scene, PicError, load, map_stats, render_static, static_status, probe_fill, probe_ffma, EXPORTS, OPT_BRUTE_FORCE, OPT_DEPTH32, OPT_COUNTERS, OPT_VIEW_FIRST,
                      OPT_VIEW_COUNT, OPT_TIMING, OPT_DEBUG_FLAGS, OPT_OUT_RELATIVE, OPT_OCCLUSION, FLAG_NONFINITE_POSE, FLAG_COLOUR_INCOMPLETE, FLAG_COLOUR_FRAGMENTS)

__all__ = ["Scene", "PicError", "load", "map_stats", "render_static", "static_status", "probe_fill", "probe_ffma", "build", "EXPORTS", "OPT_BRUTE_FORCE", "OPT_DEPTH32", "OPT_COUNTERS",
           "OPT_VIEW_FIRST", "OPT_VIEW_COUNT", "OPT_TIMING", "OPT_DEBUG_FLAGS", "OPT_OUT_RELATIVE", "OPT_OCCLUSION", "FLAG_NONFINITE_POSE", "FLAG_COLOUR_INCOMPLETE", "FLAG_COLOUR_FRAGMENTS"]
