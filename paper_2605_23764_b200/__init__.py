"""B200-native Dispatch->Combine MoE-FFN layer (forward + backward) behind a C ABI.

`binding` mirrors include/moe_b200.h call for call; `MoeLayer` is a small convenience wrapper.
The CUDA library must have been built (python -m paper_2605_23764_b200.build); nothing here
falls back to another implementation.
"""
from .binding import (MOE_BUF, MOE_FLAG_RENORM_TOPK, MOE_FLAG_SAVE_FOR_BWD, MOE_FLAG_SERIAL_LAUNCH,  # noqa: F401
                      MoeError, MoeLayer, lib_path, load_library, moe_create, moe_debug_buffer, moe_destroy,
                      moe_ffn_bwd, moe_ffn_bwd_host, moe_ffn_fwd, moe_ffn_fwd_host, moe_get_phase_ms, moe_get_status,
                      moe_last_launch_count, moe_layout, moe_layout_noalloc, moe_route, moe_route_host, moe_router_bwd, moe_router_fwd, moe_set_profiling,
                      moe_sched_study, moe_sched_study_stats, moe_sched_study_workspace_bytes,
                      moe_set_wait_budget_ms, moe_strerror,
                      moe_workspace_bytes)
