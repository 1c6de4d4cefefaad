"""prepack-b200: prefill attention over bin-packed prompts on NVIDIA B200 (sm_100a).

Thin Python binding over the C-ABI library declared in ``include/pp.h``; every step of
the path (packing, restart rotary encoding, packed attention, KV unpack) runs inside that
library. PyTorch is used by callers only for device memory and streams.
"""
from .binding import (PP_FLAG_KEEP_ROPE_TABLE, PP_FLAG_ROPE_ONLY, PP_FLAG_SKIP_ROPE, AttnParams, Packing, PrepackError,
                      Workspaces, lib_path, load_library, pp_decode_step, pp_decode_workspace_bytes,
                      pp_fill_position_ids,
                      pp_last_cuda_error, pp_pack, pp_prefill_attention, pp_prefill_fused,
                      pp_prefill_fused_host_bytes, pp_prefill_fused_workspace_bytes, pp_prefill_host,
                      pp_prefill_host_arena_bytes, pp_prefill_host_groups, pp_prefill_schedule_info, pp_prefill_workspace_bytes, pp_selftest_bounded_wait, pp_strerror,
                      pp_unpack_kv, pp_unpack_kv_static, pp_unpack_static_max_prompts,
                      pp_unpack_workspace_bytes, pp_version)

__all__ = [
    "PP_FLAG_KEEP_ROPE_TABLE", "PP_FLAG_ROPE_ONLY", "PP_FLAG_SKIP_ROPE", "AttnParams", "Packing", "PrepackError", "Workspaces",
    "lib_path", "load_library", "pp_decode_step", "pp_decode_workspace_bytes", "pp_fill_position_ids", "pp_last_cuda_error", "pp_pack",
    "pp_prefill_attention", "pp_prefill_fused", "pp_prefill_fused_host_bytes", "pp_prefill_fused_workspace_bytes", "pp_prefill_host", "pp_prefill_host_arena_bytes",
    "pp_prefill_host_groups", "pp_prefill_schedule_info",
    "pp_prefill_workspace_bytes", "pp_selftest_bounded_wait", "pp_strerror", "pp_unpack_kv", "pp_unpack_kv_static",
    "pp_unpack_static_max_prompts", "pp_unpack_workspace_bytes",
    "pp_version",
]
