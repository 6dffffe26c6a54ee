"""B200 (sm_100a) library for HMAR's Markovian block-sparse attention: Python binding.

The product is the C-ABI shared library built from csrc/ (see include/hmar.h); this package
only loads it and marshals torch device buffers into its calls.
"""
from .binding import (  # noqa: F401
    HMAR_ERR_BAD_ARG, HMAR_ERR_BOUNDS, HMAR_ERR_CUDA, HMAR_ERR_DEVICE_TIMEOUT, HMAR_ERR_UNSUPPORTED,
    HMAR_ERR_WORKSPACE, HMAR_OK, HMAR_WINDOW_CAUSAL, HMAR_WINDOW_MARKOV, HMAR_WINDOW_PREV, HMAR_WINDOW_SELF, EXPORTED_SYMBOLS, HmarError, hmar_attn_bwd, hmar_attn_bwd_noalloc, HMAR_NOALLOC_MAX_ROWS,
    hmar_attn_bwd_workspace_bytes, hmar_attn_fwd, hmar_attn_fwd_packed, hmar_attn_bwd_packed, hmar_attn_scale_step, hmar_attn_scale_step_strided, hmar_debug_force_simt,
    hmar_device_status, hmar_launch_count, hmar_profile_begin, hmar_profile_end, hmar_recon_accumulate, hmar_recon_downsample, hmar_schedule_bwd_full_tile_share, hmar_schedule_tiles, hmar_selftest_bounded_wait, hmar_shutdown, lib, status_string,
)
