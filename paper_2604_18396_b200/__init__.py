"""B200 (sm_100a) early-exit decode library: thin Python binding over the C ABI in include/river.h."""
from .binding import (argmax_noalloc, RIVER_EXIT_BATCH_MIN, RIVER_EXIT_PER_TOKEN, RIVER_F_GRAPH, RIVER_F_NO_TC, River, RiverError,
                      make_config, river_config)
from .buildlib import build

__all__ = ["River", "argmax_noalloc", "RiverError", "make_config", "river_config", "build", "RIVER_EXIT_PER_TOKEN",
           "RIVER_EXIT_BATCH_MIN", "RIVER_F_GRAPH", "RIVER_F_NO_TC"]
