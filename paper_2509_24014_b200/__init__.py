"""SparseD attention hot path for NVIDIA B200: C-ABI CUDA library plus a thin ctypes binding."""
from .binding import (  # noqa: F401
    MODE_FULL, MODE_FULL_AND_SELECT, MODE_SPARSE, VARIANT_NO_REUSE, VARIANT_NO_ISOLATION, OP_ATTN_FULL, OP_ATTN_SPARSE, OP_PATTERN_VALIDATE,
    OP_SELECT_FROM_SCORES, OP_SELECT_PATTERN, OP_SELECT_POOLED_QK, OP_ATTENTION_STEP, Pattern, SelectParams, Shape, SparsedError, load_library,
    make_params, make_shape, new_pattern, new_tile_stats, sparsed_attn_full_stats, sparsed_select_from_stats,
    sparsed_tile_stats_bytes, new_workspace, pattern_from_csr, sparsed_attn_full, sparsed_attn_sparse, sparsed_attention_step, sparsed_attention_step_variant,
    sparsed_build_window_pattern,
    sparsed_kept_per_row, sparsed_last_device_status, sparsed_pattern_validate, sparsed_schedule_mode,
    sparsed_select_from_scores, sparsed_select_pattern, sparsed_select_pattern_pooled_qk, sparsed_select_pattern_static, sparsed_switch_step, sparsed_workspace_bytes,
    sparsed_workspace_init, sparsed_selftest_wait_timeout, save_pattern, load_pattern,
)
