"""B200-native (sm_100a) late-interaction retrieval: thin Python binding over libchimera's C ABI.

Every step of a search runs in the CUDA library; this package only marshals arguments (torch tensors supply device
memory and the stream).  There is no CPU fallback: importing the binding without the built library fails loudly.
"""
from .binding import (ChimeraError, GraphedSearch, Index, Taps, lib, library_path, probes_static, profile_enable, profile_read,  # noqa: F401
                      PROFILE_SLOTS)
from .sharded import ShardEngine, ShardedSearcher, all_gather_stack, shard_ranges  # noqa: F401
