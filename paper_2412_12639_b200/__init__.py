"""B200 (sm_100a) implementation of the tree-verification step of Falcon
speculative decoding: tree-masked attention, greedy acceptance and KV compaction
behind the C ABI of include/falcon.h.

`binding` is the ctypes layer over libfalcon.so (loaded on first use; missing
library = error, never a fallback).  `synth` draws seeded synthetic inputs and
is independent of the library.
"""
from . import binding, synth  # noqa: F401
from .binding import (ATTN_AUTO, ATTN_SIMT, ATTN_TC, Context, FalconError, accept_args, attn_args,  # noqa: F401
                      compact_args, topm_args, tree_desc)
