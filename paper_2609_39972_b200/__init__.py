"""B200-native (sm_100a) draft-tree + verification hot path of UBTree, behind the C ABI of include/ubt.h.

``binding`` holds thin ctypes wrappers with the names of the C entry points; the CUDA library itself
is ``libubt.so`` next to this file, built by ``_build.build()``.
"""
from .binding import (Tree, ubt_debug_ring_timeouts, UbtError, VerifyResult, load, status_string, ubt_build_mask, ubt_build_tree, ubt_selector_scores,
                      ubt_draft_host_buffer_bytes, ubt_draft_tree, ubt_draft_tree_host, ubt_draft_workspace_bytes,
                      ubt_topk_logprob, ubt_topk_shard, ubt_topk_shard_bytes, ubt_topk_merge_shards, gather_shard_partials, topk_logprob_vocab_parallel, verify_tree_vocab_parallel, ubt_verify_keys_shard, ubt_verify_tree_keys, ubt_verify_tree_picks, verify_tree_from_hidden, verify_tree_from_hidden_vocab_parallel, ubt_sample_totals_shard, ubt_sample_picks_shard, sample_tree_vocab_parallel, ubt_lm_head_topk, ubt_lm_head_topk_shard, lm_head_topk_vocab_parallel, ubt_lm_head_workspace_bytes, ubt_verify_host_buffer_bytes, ubt_verify_tree, ubt_verify_tree_host, ubt_verify_tree_static, ubt_verify_static_capacity,
                      ubt_verify_workspace_bytes, ubt_version, workspace)

__all__ = [n for n in dir() if n.startswith("ubt_")] + ["Tree", "VerifyResult", "UbtError", "load", "status_string",
                                                       "workspace"]
