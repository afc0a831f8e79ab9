"""Slim-DP communication round on B200: thin Python binding of the C ABI in
include/slimdp.h.  Every step runs in the CUDA library; this package only
marshals torch tensors (device pointers, sizes, the current stream)."""
from .binding import (explore_shard_workspace_bytes, slimdp_sample_explore_shard, select_segmented_workspace_bytes, slimdp_select_core_segmented, Q8_BUCKET, slimdp_pack_q8_batched, slimdp_merge_q8, slimdp_select_shard_begin, slimdp_select_hist, slimdp_select_resolve, slimdp_select_count, slimdp_select_emit, WIRE_KEYS_WANTED, slimdp_wire_pack, slimdp_wire_unpack, wire_message_bytes, wire_read_status, RoundContext, SlimDPError, release_default_round_ctx, round_stage_bytes, core_aux_bytes, core_aux_dir_offset, explore_workspace_bytes, launch_count, lib, mark_dominant_kernel,
                      read_status, round_arena_bytes, select_workspace_bytes, slimdp_core_signature, wire_bytes, slimdp_dense_merge_score, slimdp_exchange, slimdp_merge, slimdp_pack,
                      slimdp_pack_batched, slimdp_pull, slimdp_pull_batched, slimdp_round, slimdp_round_host,
                      slimdp_sample_explore, slimdp_sample_explore_batched, slimdp_sample_explore_static,
                      slimdp_worker_merge_batched, slimdp_score, slimdp_select_core,
                      workspace_bytes)
from .driver import SlimDPDriver
from .sharded import CudaBackend, select_core_sharded, shard_bounds, tie_quotas
from .round import RoundBuffers, run_round

__all__ = [
    "explore_shard_workspace_bytes", "slimdp_sample_explore_shard", "select_segmented_workspace_bytes", "slimdp_select_core_segmented", "Q8_BUCKET", "slimdp_pack_q8_batched", "slimdp_merge_q8", "CudaBackend", "select_core_sharded", "shard_bounds", "tie_quotas",
    "slimdp_select_shard_begin", "slimdp_select_hist", "slimdp_select_resolve", "slimdp_select_count", "slimdp_select_emit",
    "WIRE_KEYS_WANTED", "slimdp_wire_pack", "slimdp_wire_unpack", "wire_message_bytes", "wire_read_status", "RoundContext", "release_default_round_ctx", "round_stage_bytes", "SlimDPError", "lib", "launch_count", "mark_dominant_kernel", "core_aux_bytes", "core_aux_dir_offset", "select_workspace_bytes",
    "explore_workspace_bytes", "workspace_bytes", "round_arena_bytes", "read_status", "slimdp_score",
    "slimdp_select_core", "slimdp_sample_explore", "slimdp_sample_explore_batched", "slimdp_sample_explore_static", "slimdp_pack",
    "slimdp_core_signature", "wire_bytes", "slimdp_pack_batched", "slimdp_exchange", "slimdp_dense_merge_score", "slimdp_worker_merge_batched", "slimdp_merge", "slimdp_pull", "slimdp_pull_batched", "slimdp_round", "slimdp_round_host",
    "RoundBuffers", "run_round", "SlimDPDriver",
]
