"""B200-native per-chunk KV-cache codec: thin Python binding over the C ABI in include/kvh.h.

Every step of the path runs in the CUDA kernels of ``libkvh.so``; this package
only marshals arguments (tensor pointers, the current CUDA stream).  There is no
CPU fallback: calling into the library without the built extension raises.
"""
from .binding import (  # noqa: F401
    CHUNK_TOKENS, GROUP, NUM_LEVELS, ChunkDesc, KvhError, Pool, decode_batch, decode_to_pages,
    descs_to_tensor, encode, encode_chunks, format_version, level_bytes, level_info, lib, load_host,
    load_host_static, plan_chunks, keep_sinks_and_recent, encode_kept, RUN_DTYPE, transcode, check_page_table, policy_assign, policy_assign_tiers, OPTION_DTYPE, TIER_DTYPE, status_string, store_host, STATIC_STAGING_BYTES,
)
