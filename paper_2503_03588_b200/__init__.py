"""PowerAttention block-sparse attention for NVIDIA B200 (sm_100a): Python face of the C ABI.

The CUDA library is required; importing the package without it raises ImportError.
"""
from .binding import (PA_BF16, PA_F32, PaError, pa_build_layout, pa_build_tile_layout, pa_build_window_layout, pa_reach_counts, pa_window_layout_size, pa_decode, pa_decode_block_list, pa_decode_static,
                      pa_decode_paged, pa_decode_paged_workspace_bytes, pa_decode_row_block_set, pa_decode_status, pa_kv_append,
                      pa_reload_environment, pa_set_wait_limit_cycles, pa_decode_workspace_bytes, pa_layout_size, pa_prefill, pa_prefill_varlen, pa_prefill_backward, pa_prefill_status,
                      pa_prefill_workspace_bytes, pa_status_string, pa_tile_layout_size, pa_version)

__all__ = ["PA_BF16", "PA_F32", "PaError", "pa_build_layout", "pa_build_tile_layout", "pa_build_window_layout", "pa_reach_counts", "pa_window_layout_size", "pa_decode", "pa_decode_block_list", "pa_decode_static",
           "pa_decode_paged", "pa_decode_paged_workspace_bytes", "pa_decode_row_block_set", "pa_decode_status", "pa_kv_append",
           "pa_reload_environment", "pa_set_wait_limit_cycles", "pa_decode_workspace_bytes", "pa_layout_size", "pa_prefill", "pa_prefill_varlen", "pa_prefill_backward", "pa_prefill_status",
           "pa_prefill_workspace_bytes", "pa_status_string", "pa_tile_layout_size", "pa_version"]
