"""RBS-Attention prefill hot path for NVIDIA B200: block statistics, dual-branch block selection and
causal block-sparse attention as hand-written sm_100a kernels behind a small C ABI (include/rbs.h).

The Python names mirror the C entry points.  Importing this package does not load the CUDA library;
the first call does, and raises if it has not been built.
"""
from .binding import (BlockStats, RbsError, alloc_stats, load_library, rbs_block_stats, rbs_block_stats_box, rbs_device_status, rbs_select_box,
                      rbs_mask_group_union, rbs_select, rbs_select_chunk, rbs_select_static, rbs_sparse_prefill_chunk, rbs_sparse_prefill, rbs_sparse_prefill_grouped, workspace_bytes)

__all__ = ["BlockStats", "RbsError", "alloc_stats", "load_library", "rbs_block_stats", "rbs_block_stats_box", "rbs_device_status", "rbs_select_box",
           "rbs_mask_group_union", "rbs_select", "rbs_select_chunk", "rbs_select_static", "rbs_sparse_prefill_chunk", "rbs_sparse_prefill", "rbs_sparse_prefill_grouped", "workspace_bytes"]
