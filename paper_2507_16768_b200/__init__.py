"""B200 (sm_100a) allowed-token mask build + apply for operator-automaton structured decoding.

The product is the C-ABI library ``libwg.so`` (``include/wg.h``); this package is its thin
Python binding.  Build the library with ``python -m paper_2507_16768_b200.build``.
"""
from .binding import *  # noqa: F401,F403
from .binding import (Context, Grammar, Vocab, WgError, kernel_launch_count, wg_advance,
                      wg_apply_mask, wg_apply_workspace_bytes, wg_build_masks, wg_decode_step,
                      wg_decode_step_host, wg_mask_cache_lookup)
