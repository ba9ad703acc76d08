"""Moment-KV decode hot path for B200: thin Python binding over the C-ABI CUDA library."""
from .mkv import (  # noqa: F401
    MKV_BF16, MKV_F32, MKV_KERNEL_AUTO, MKV_KERNEL_MMA, MKV_KERNEL_SIMT, MKV_FLAG_RECORD_PROBS,
    MKV_FLAG_INPUTS_READY, MKV_FLAG_REPRODUCIBLE, MKV_OPT_RING_STAGES, MKV_OPT_HEAD_TILES, MKV_OPT_WAIT_LIMIT_US,
    MKV_OPT_OVERLAP, MKV_OPT_GRID_SHARE, MKV_INJECT_LOST_TILE, grid_limit, plan_ranges,
    MKV_SCORE_GROUP_MEAN, MKV_SCORE_LAYER_MEAN, MkvError, MomentKV, load_library, workspace_bytes,
    kv_bytes_per_token, status_string, EXPORTED_SYMBOLS, attend_noalloc, plan_starts,
)
