"""Lory MoE layer (causal segment routing + expert merging) for NVIDIA B200.

`binding` mirrors the C ABI declared in include/lory.h; `workloads` holds the seeded
synthetic inputs; `build` compiles the CUDA library in-tree.
"""
from . import binding, workloads  # noqa: F401
from .binding import (LORY_BF16, LORY_FLAG_ACCUMULATE_GRADS, LORY_FLAG_CHUNKED_ADJOINT, LORY_FLAG_FIRST_SEGMENT_GRAD, LORY_FLAG_PREFIX_ROUTING, LORY_FLAG_REUSE_MERGED, LORY_FLAG_SIMT, LORY_FP32, LoryError, lory_check_status, lory_dims,  # noqa: F401
                      lory_expert_utilization,
                      lory_last_launch_count, lory_moe_backward, lory_moe_ffn, lory_profile_enable, lory_profile_read, lory_route_noalloc, lory_selftest_bounded_wait, lory_moe_forward,
                      lory_block_backward, lory_block_forward, lory_block_workspace_bytes,
                      lory_moe_step_host, lory_moe_step_host_bytes, lory_moe_step_host_enqueue,
                      lory_moe_step_host_pipeline_bytes, lory_moe_step_host_wait, lory_moe_workspace_bytes,
                      lory_status_string, make_dims)
