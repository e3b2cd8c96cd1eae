"""B200-native tree draft-and-verify step of VADUSA (speculative decoding with a
tolerance rule for a VALL-E-style speech-token language model).

The work is done by libvadusa.so (hand-written CUDA for sm_100a behind a C
ABI, see include/vadusa.h); this package only marshals arguments.  There is no
CPU path: without the compiled library, or without a B200, calls fail.
"""
from .binding import (Config, Sampling, Stats, Vadusa, VadusaError, lib, load_library, pack_weights,
                      tensor_infos, MAX_PATH, draft_topk_static, build_sparse_tree)

__all__ = ["Config", "Sampling", "Stats", "Vadusa", "VadusaError", "lib", "load_library", "pack_weights",
           "tensor_infos", "MAX_PATH", "draft_topk_static", "build_sparse_tree"]
