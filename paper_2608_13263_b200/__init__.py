"""B200-native repack path of vToken: compaction of the live tokens of a token-evicted paged
KV cache into dense blocks with rewritten block and token tables.

The work is done by hand-written CUDA kernels (sm_100a) behind the C ABI declared in
``include/vtoken.h``; this package is the thin Python binding of that ABI (same function
names, argument marshalling only).  There is no CPU fallback: using the binding without the
built library raises ImportError.
"""
from .binding import (  # noqa: F401
    VtokenError,
    vtoken_apply_moves,
    vtoken_block_liveness,
    vtoken_check_tables,
    vtoken_digest_logical,
    vtoken_plan_partial,
    vtoken_build_slot_mapping,
    vtoken_evict_tokens,
    vtoken_evict_tokens_counted,
    vtoken_sync_new_tokens,
    vtoken_sync_new_tokens_counted,
    vtoken_copy_grid,
    vtoken_create,
    vtoken_destroy,
    vtoken_gather_logical,
    vtoken_gather_logical_noalloc,
    vtoken_plan,
    vtoken_read_counts,
    vtoken_repack,
    vtoken_repack_host,
    vtoken_repack_host_partial,
    vtoken_repack_waves,
    vtoken_slot_cache_mark,
    vtoken_slot_cache_update,
    vtoken_waves_workspace_bytes,
    vtoken_scratch_bytes,
)

__all__ = ["VtokenError", "vtoken_create", "vtoken_destroy", "vtoken_plan", "vtoken_repack",
           "vtoken_gather_logical", "vtoken_read_counts", "vtoken_repack_host", "vtoken_copy_grid",
           "vtoken_scratch_bytes", "vtoken_gather_logical_noalloc", "vtoken_evict_tokens", "vtoken_sync_new_tokens",
           "vtoken_build_slot_mapping", "vtoken_apply_moves", "vtoken_block_liveness", "vtoken_plan_partial", "vtoken_digest_logical",
           "vtoken_repack_host_partial", "vtoken_repack_waves", "vtoken_waves_workspace_bytes", "vtoken_slot_cache_mark",
           "vtoken_slot_cache_update", "vtoken_check_tables", "vtoken_evict_tokens_counted",
           "vtoken_sync_new_tokens_counted"]
