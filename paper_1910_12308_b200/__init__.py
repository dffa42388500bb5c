"""B200-native SwarmSGD pairwise-gossip interaction path (hand-written CUDA for sm_100a behind a C ABI)."""
from .binding import (BLOCKING, NONBLOCKING, OBJ_LSQ, OBJ_NONE, OBJ_SYNTH, BF16, F32, Swarm, SwarmError, load,
                      library_path)

__all__ = ["Swarm", "SwarmError", "load", "library_path", "BLOCKING", "NONBLOCKING", "OBJ_NONE", "OBJ_SYNTH",
           "OBJ_LSQ", "F32", "BF16"]
