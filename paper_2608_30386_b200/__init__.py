"""B200-native hot path of Decay-Aware State Compression (DASC): plan, pack,
restore (zero-fill) and suffix refresh of linear-attention state checkpoints.

All compute runs in ``libdasc.so`` (hand-written sm_100a CUDA behind a C ABI,
declared in ``include/dasc.h``); this package only marshals arguments.
"""
from .binding import (  # noqa: F401
    ALGO_AUTO, ALGO_CHUNKED, ALGO_SEQUENTIAL, GDN, IO_BF16, IO_FP32, KDA, REFRESH_CONTINUE,
    REFRESH_SCRATCH_MERGE_LOCAL, SCOPE_HEAD, SCOPE_LAYER, SCOPE_MODEL, SEL_EXPLICIT, SEL_THRESHOLD, SEL_TOP_RATIO,
    DascError, Plan, dasc_pack, dasc_plan, dasc_refresh, dasc_refresh_static, dasc_refresh_status, dasc_refresh_window, dasc_refresh_workspace_bytes,
    dasc_int8_slot_bytes, dasc_pack_int8, dasc_restore, dasc_restore_int8, lib, status_string, version,
    LAYOUT_DENSE, LAYOUT_PADDED, LAYOUT_RAGGED, dasc_checkpoint_bytes, dasc_pack_padded, dasc_padded_pool_floats,
    dasc_restore_padded, dasc_slot_budget, dasc_tp_balance, dasc_pack_tp, dasc_restore_tp, dasc_tp_head_permutation,
    dasc_conv_store, dasc_conv_load, dasc_plan_save, dasc_plan_load, dasc_refresh_counters, dasc_debug_set_refresh_poll_limit,
)
