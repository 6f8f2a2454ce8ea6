"""ParallelComp attention hot path for B200 (sm_100a): thin Python binding over libpc.so.

The functions here only marshal arguments (torch tensors -> device pointers); every
step of the path runs in the CUDA kernels behind the C ABI declared in include/pc.h.
There is no CPU fallback: importing :mod:`paper_2502_14317_b200.binding` raises if the
library is missing.
"""
from .binding import (  # noqa: F401
    PcError, lib_path, load_library, version, status_string, launch_count,
    chunk_prefill_attn, chunk_prefill_attn_workspace_bytes, chunk_score_from_lse, rope_position_reuse,
    select_chunks, score_select_chunks, select_tokens, select_tokens_calibrated, gather_kv, parallel_attn, parallel_attn_append, parallel_attn_workspace_bytes,
    parallel_attn_static, parallel_attn_static_scratch_bytes, hot_path, hot_path_from_host,
    queue_init, queue_update, queue_gather, queue_select_gather, queue_emit, hot_path_streaming,
)
