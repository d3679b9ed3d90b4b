"""LAVa prefill-time KV-cache eviction hot path for B200 (sm_100a).

Thin ctypes binding over liblava.so (hand-written CUDA).  The functions below carry the names
of the C ABI in include/lava.h and only marshal arguments: every step runs in the library's
kernels.  There is no CPU or PyTorch fallback; a missing library raises at first use.
"""
from .binding import (  # noqa: F401
    LAVA_BF16, LAVA_F32, LAVA_POOL_AVG, LAVA_POOL_MAX, LAVA_POOL_NONE,
    LAVA_BUDGET_DYNAMIC, LAVA_BUDGET_UNIFORM, LAVA_BUDGET_PYRAMID,
    LAVA_FLAG_PER_HEAD_TOPK, LAVA_FLAG_UNIT_VALUE_NORM, LAVA_FLAG_TOKEN_VALUE_NORM,
    LavaError, LayerDesc, library_path, load_library,
    lava_version, lava_last_error, lava_workspace_bytes, lava_poll_status, lava_wo_norm,
    lava_score_layer, lava_score_layer_static, lava_score_layers, lava_layer_budgets,
    lava_select_topk, lava_select_topk_layers, lava_compact_kv, lava_compact_kv_layers,
    EvictionPlan, evict_model, lava_layer_output_loss,
    lava_select_shard_bytes, lava_select_shard_layout, lava_select_shard_begin, lava_select_shard_hist,
    lava_select_shard_step, lava_select_shard_count, lava_select_shard_emit,
    lava_decode_workspace_bytes, lava_decode_attention_layers, lava_decode_attention, Cascade, lava_cascade_state_bytes,
    lava_launch_count, lava_score_path, lava_set_option, lava_get_option, lava_host_arena_bytes, lava_evict_model_host,
)
