"""B200 (sm_100a) hot path of dynamic-width speculative beam decoding: forest-masked attention
and the verification step, as a C-ABI CUDA library with a thin binding of the same names."""
from .binding import (Forest, DsbdError, forest_attention, forest_attention_workspace, forest_attention_launches,  # noqa: F401
                      verify_step, verify_workspace, alloc_verify_out, default_out_off, select_width, node_stats, node_stats_static, kv_commit, draft_layer, forest_attention_paged, kv_commit_paged, forest_build,
                      status_string, load, lib_path)
