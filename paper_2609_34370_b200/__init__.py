"""B200-native speculative-decoding verify step: a ctypes binding over libspx.so.

The binding only marshals arguments (torch tensors -> device pointers, sizes, the current CUDA
stream); every step of the path runs in the library's CUDA kernels.  There is no CPU fallback:
importing the binding's functions without the compiled library, or calling them with host
tensors, raises.
"""
from .binding import (  # noqa: F401
    SpxError, Workspace, exported_symbols, lib_path, load_library, rejection_sample, verify_attention,
    verify_step, verify_step_host, workspace_size, DEV_BAD_PAGE, DEV_BAD_TOKEN, DEV_BAD_LEN, DEV_TIMEOUT,
    DEV_DEGENERATE, DEV_BAD_PARAM, last_launch_count, plan_layout, debug_timeline, set_timing_events, host_step_arena_size,
    make_attn_args, make_sample_args, rejection_sample_static, STATIC_SCRATCH_BYTES, kv_append, kv_rollback, draft_confidence, select_speculation, lookahead_memory, sp_effective_batch, selective_batch,
    selective_effective_batch, delay_gain, lm_head,
)
