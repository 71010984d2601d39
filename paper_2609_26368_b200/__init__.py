"""B200-native hybrid sparse attention hot path of HySparse2 (C-ABI library + thin Python binding)."""
from . import binding
from .binding import (HS2Error, Problem, hs2_device_error_flags, hs2_full_attn_select, hs2_full_attn_select_fp8kv, hs2_kv_project, hs2_kv_project_fp8_records, hs2_launch_count, hs2_probe_gather,
                      hs2_set_filter_min_keys, hs2_set_tcgen05_enabled, hs2_sparse_attn_decode,
                      hs2_sparse_attn_decode_fp8kv, hs2_sparse_attn_decode_static, hs2_sparse_attn_prefill,
                      hs2_sparse_attn_prefill_fp8kv, hs2_status_string, hs2_topk_select, hs2_workspace_bytes,
                      library_path, load_library)

__all__ = ["HS2Error", "Problem", "binding", "hs2_device_error_flags", "hs2_full_attn_select", "hs2_full_attn_select_fp8kv", "hs2_kv_project", "hs2_kv_project_fp8_records", "hs2_launch_count", "hs2_probe_gather",
           "hs2_set_filter_min_keys", "hs2_set_tcgen05_enabled", "hs2_sparse_attn_decode", "hs2_sparse_attn_decode_fp8kv",
           "hs2_sparse_attn_decode_static", "hs2_sparse_attn_prefill", "hs2_sparse_attn_prefill_fp8kv",
           "hs2_status_string", "hs2_topk_select", "hs2_workspace_bytes", "library_path", "load_library"]
