"""B200-native batch-1 decode step of a Qwen2.5-style decoder behind a C ABI (libedgefm.so).

The Python layer only marshals arguments (ctypes) and uses torch for device memory and streams;
every step of the computation runs in the hand-written sm_100a kernels of csrc/.
"""
from .binding import (EdgefmError, Status, edgefm_create, edgefm_decode_step, edgefm_destroy, edgefm_export_kv,
                      edgefm_get_length, edgefm_get_launches_per_step, edgefm_last_error, edgefm_prefill_kv,
                      edgefm_version, edgefm_sync_status, edgefm_debug_profile, edgefm_debug_set_wait_limit, edgefm_debug_set_prefill_wait, edgefm_debug_prefill_plan, edgefm_debug_plan, edgefm_debug_plan_operator, edgefm_decode_step_static, edgefm_set_vocab_subset, edgefm_append_kv, edgefm_export_kv_int8, edgefm_verify_block, edgefm_sync_length, edgefm_prefill_tokens, edgefm_prefill, library_path, load_library, DecodeContext, upload_weights)

__all__ = ["EdgefmError", "Status", "edgefm_create", "edgefm_decode_step", "edgefm_destroy", "edgefm_export_kv",
           "edgefm_get_length", "edgefm_get_launches_per_step", "edgefm_last_error", "edgefm_prefill_kv",
           "edgefm_version", "edgefm_sync_status", "edgefm_debug_profile", "edgefm_debug_set_wait_limit", "edgefm_debug_set_prefill_wait", "edgefm_debug_prefill_plan", "edgefm_debug_plan", "edgefm_debug_plan_operator", "edgefm_decode_step_static", "edgefm_set_vocab_subset", "edgefm_append_kv", "edgefm_export_kv_int8", "edgefm_verify_block", "edgefm_sync_length", "edgefm_prefill_tokens", "edgefm_prefill", "library_path", "load_library", "DecodeContext", "upload_weights"]
