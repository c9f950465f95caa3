"""B200-native FP8-KV decode attention (split-KV + merge) and fused FP8 KV append.

The compute runs in ``lib/libpuzzle_attn.so`` (hand-written sm_100a kernels behind a C ABI,
declared in ``include/puzzle_attn.h``).  This package only marshals torch tensors into that
ABI; there is no Python or CPU fallback: a missing library raises.
"""
from .binding import (  # noqa: F401
    KV_BF16,
    KV_FP8_E4M3,
    DEV_BAD_BLOCK,
    DEV_SEQ_TOO_LONG,
    DEV_WAIT_EXPIRED,
    STATIC_SCRATCH_BYTES,
    SCHED_AUTO,
    SCHED_CTA,
    SCHED_WARP,
    KVView,
    LayerDesc,
    PuzzleError,
    calibrate_scales,
    kv_view,
    layer_desc,
    library_path,
    puzzle_attn_merge,
    puzzle_attn_merge_strided,
    puzzle_decode_attn,
    puzzle_decode_attn_partial,
    puzzle_decode_attn_static,
    puzzle_decode_attn_tcgen05,
    puzzle_decode_attn_tokens,
    puzzle_decode_attn_tokens_workspace_bytes,
    puzzle_decode_attn_tokens_workspace_init,
    puzzle_decode_attn_workspace_bytes,
    puzzle_decode_step_host,
    puzzle_decode_step_host_staging_bytes,
    puzzle_decode_attn_workspace_init,
    puzzle_hbm_read_probe,
    puzzle_kv_amax_update,
    puzzle_kv_append,
    puzzle_kv_append_tokens,
    puzzle_kv_scales_from_amax,
    puzzle_launch_count,
    puzzle_decode_attn_kernel_name,
    puzzle_status_string,
)
from .stack import DecodeStack  # noqa: F401,E402
from .paging import cache_blocks, linear_block_table, multi_token_args, ring_block_table, window_ring_blocks  # noqa: F401,E402
from .parallel import ContextShardedAttention, context_slice, head_slice  # noqa: F401,E402
