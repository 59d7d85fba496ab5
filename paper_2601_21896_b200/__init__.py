"""PaFu-KV inference hot path for NVIDIA B200: score -> select -> compact -> chunk attention.

The product is the C-ABI CUDA library ``libpafu.so`` (see ``include/pafu.h``); this package is
its thin Python binding plus the seeded workload generator.  Nothing here computes on the CPU.
"""
from .binding import (  # noqa: F401
    ACT_GELU, ACT_SILU, FINAL_NONE, FINAL_SIGMOID, PafuError, Shape, Head, make_policy,
    pafu_version, pafu_kept_counts, pafu_workspace_bytes, pafu_workspace_status, pafu_workspace_counters, pafu_score, pafu_score_qkv,
    pafu_select, pafu_compact, pafu_compact_layers, pafu_cache_update, Cache, pafu_chunk_attn, pafu_chunk_attn_indexed, pafu_chunk_attn_noalloc, pafu_step, pafu_step_indexed,
    pafu_step_host, pafu_step_host_async,
    pafu_step_host_arena_bytes, pafu_sse, pafu_sse_mean_first, pafu_sse_workspace_bytes, pafu_step_timed, event_handles, step_args, lib,
)
