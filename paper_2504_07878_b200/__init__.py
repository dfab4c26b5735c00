"""Token-level routing step for B200: Python binding of the C-ABI library libtlr.so."""
from .binding import (TLR_DEV_NONFINITE, TLR_DEV_WAIT_TIMEOUT, TLR_OK, TLR_PATH_AUTO, TLR_PATH_SIMT, TLR_PATH_TC, TLR_SCORE_CONF, TLR_SCORE_MLP, TLR_STATIC_MAX_ROWS,
                      Router, TlrError, TlrPlan, TlrRouteOptions, load_library, status_string, tlr_create, tlr_create_fp8, tlr_debug_inject, tlr_debug_plan_tiles, tlr_destroy,
                      tlr_last_device_status, tlr_plan_query, tlr_read_kernel_timing, tlr_route, tlr_route_ex, tlr_route_host, tlr_route_host_collect, tlr_route_host_submit, tlr_route_static,
                      tlr_set_kernel_timing, tlr_set_path, tlr_set_router_mlp, tlr_shard_finish, tlr_shard_summary,
                      tlr_debug_shard_table, tlr_rows_merge, tlr_shard_attach, tlr_shard_block_bytes, tlr_shard_finish_fused, tlr_shard_push)
from .sharded import (FusedVocabShardedRouter, VocabShardedRouter, exchange_routed, gather_summaries, merge_routed,
                      row_offsets, shard_bounds, symmetric_exchange_block)
