"""B200-native cached neighbour sampling (GraphSnapShot's GraphSDSampler hot path).

Thin ctypes binding over the C-ABI CUDA library ``libgs.so`` (see ``include/gs.h``); every
step of the path runs in that library's kernels.  There is no CPU fallback: if the library is
missing or cannot be loaded, importing :mod:`paper_2406_17918_b200.binding` raises.
"""
from .binding import (  # noqa: F401
    GS_MODE_FCR, GS_MODE_OTF, GS_MODE_FBL, GS_MODE_OTF_FETCH, GS_F32, GS_BF16, GsError, Block, Graph, Cache,
    gs_graph_create, gs_graph_validate, gs_graph_set_gather_grid, gs_cache_bytes, gs_workspace_bytes, gs_cache_init, gs_cache_refresh_all, gs_cache_bytes_split, gs_graph_count_dense, gs_cache_init_split, gs_sample_batch,
    gs_sample_batch_host, gs_sample_batch_noalloc, NOALLOC_SCRATCH_BYTES, gs_batch_counts, gs_gather_features, gs_cache_read_rows, gs_gather_rows, gs_gather_rows_peer, gs_shard_bucket, gs_shard_workspace_bytes, gs_shard_sample_rows, gs_shard_status, gs_shard_extend, gs_shard_merge, gs_shard_fan_out, gs_gather_status,
    gs_cache_export, gs_cache_import, gs_sync_status, gs_batch_stats, gs_cache_profile_begin, gs_cache_profile_end, gs_cache_set_tuning, gs_debug_set_grid_cap, gs_kernel_launches, gs_alu_ceiling, gs_cache_set_dedup, GS_DEDUP_DIRECT, GS_DEDUP_HASH, GS_DEDUP_SORT, GS_DEDUP_AUTO,
    gs_last_error, gs_stats_word_offset, library_path, exported_symbols, COUNTS_READBACK_BYTES,
)
