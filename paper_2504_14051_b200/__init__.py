"""B200-native CAOTE eviction-scoring attention step (C-ABI CUDA library + thin ctypes binding)."""
from .binding import (  # noqa: F401
    OPT_DECODE_CLUSTER, OPT_SIDE_BY_SIDE, OPT_WAIT_CYCLES, CaoteError, Params, alloc_workspace, caote_append, caote_compact, caote_launch_count, caote_post_evict_output, caote_post_evict_output_ws, caote_read_status,
    caote_score, caote_score_fast, caote_score_static, caote_score_sum_errors, caote_select_evict, caote_select_evict_greedy, caote_set_option, caote_status_string, caote_step, caote_step_fast, caote_vsum, caote_trace_collect, caote_trace_enable, caote_workspace_bytes, lib,
    library_path, make_params,
)
from .cache import EvictionCache  # noqa: F401
