"""B200 (sm_100a) HiLS attention: C-ABI CUDA library plus a thin ctypes binding.

`hils_prefill` and `hils_decode` mirror the entry points declared in include/hils.h.
The shared library is loaded on first use and there is no fallback when it is missing.
"""
from .binding import (HilsError, HilsParams, HostRunner, alloc_workspace, hils_decode, hils_decode_noalloc, hils_decode_paged, hils_decode_multi, hils_landmark_summary, hils_chunk_overlap, hils_prefill_backward, hils_attention, hils_prefill_at,
                      hils_prefill,
                      host_arena_bytes, last_launch_count, load_library, make_params, poll_status,
                      status_string, trace_enable, trace_read, version, workspace_bytes)

__all__ = ["HilsError", "HilsParams", "HostRunner", "alloc_workspace", "hils_decode", "hils_decode_noalloc", "hils_decode_paged", "hils_decode_multi", "hils_landmark_summary", "hils_chunk_overlap", "hils_prefill_backward", "hils_attention", "hils_prefill_at",
           "hils_prefill",
           "host_arena_bytes", "last_launch_count", "load_library", "make_params", "poll_status",
           "status_string", "trace_enable", "trace_read", "version", "workspace_bytes"]
