"""RoCo KV-constrained attention for one B200: Python binding of the libroco C ABI."""
from .binding import (ROCO_POLICY_H2O, ROCO_POLICY_MAS_WINDOW, ROCO_POLICY_RANDOM, ROCO_POLICY_RECENCY,
                      ROCO_POLICY_ROCO, ROCO_POLICY_SCISSORHANDS, ROCO_POLICY_STREAMLLM, ROCO_POLICY_TOVA,
                      roco_decode_step_policy, roco_prefill_blockwise, roco_decode_cluster_ranks, roco_decode_step_cluster, roco_decode_split_workspace_bytes, roco_decode_step_split,
                      EXPORTS, LIB_PATH, ROCO_ATTEND_FIRST, ROCO_BF16, ROCO_EVICT_FIRST, ROCO_F32,
                      ROCO_SCOPE_EXCLUDE_TOP_R, ROCO_SCOPE_LOWEST_R, Cache, RocoError, lib, roco_cache,
                      roco_block_step, roco_gqa_block_step, roco_prefill_blockwise_gqa, roco_consistency_step, roco_decode_host_staging_bytes, roco_decode_step, roco_gqa_decode_step, roco_decode_step_host, roco_decode_step_host_begin, roco_decode_step_host_end,
                      roco_decode_host_pipeline_staging_bytes, roco_device_status,
                      roco_prefill, roco_selftest_read_stream, roco_selftest_wait_timeout, roco_prefill_attend, roco_prefill_attend_workspace_bytes, roco_prefill_static, roco_prefill_uses_tensor_cores, roco_prefill_workspace_bytes, roco_prefill_workspace_bytes_lowest_r, status_string)
