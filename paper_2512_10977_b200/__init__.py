"""B200 (sm_100a) paged GQA decode attention: a C-ABI CUDA library and its thin Python binding.

``decode_attn`` and friends marshal torch tensors (device memory and streams only) into the
``extern "C"`` calls of ``include/decode_attn.h``; every step of the computation runs in the
library's own kernels.  There is no CPU or PyTorch fallback: if the library is missing or no
CUDA device is present, the calls raise.
"""
from .binding import (DecodeAttnError, decode_attn, decode_attn_append, decode_attn_append_fp8kv, decode_attn_cascade, decode_attn_extend, decode_attn_fp8kv, decode_attn_fp8kv_cascade, decode_attn_fp8kv_extend, decode_attn_fp8kv_extend_wide, decode_attn_fp8kv_host_io, decode_attn_host_io, decode_attn_static_scratch, ensure_workspace, get_option, timeline, use_library,
                      launch_count, lib, plan, read_device_status, set_option, version, workspace_bytes)

__all__ = ["DecodeAttnError", "decode_attn", "decode_attn_append", "decode_attn_append_fp8kv", "decode_attn_cascade", "decode_attn_extend", "decode_attn_fp8kv", "decode_attn_fp8kv_cascade", "decode_attn_fp8kv_extend", "decode_attn_fp8kv_extend_wide", "decode_attn_fp8kv_host_io", "decode_attn_host_io", "decode_attn_static_scratch", "ensure_workspace", "get_option", "timeline", "use_library",
           "launch_count", "lib", "plan", "read_device_status", "set_option", "version", "workspace_bytes"]
