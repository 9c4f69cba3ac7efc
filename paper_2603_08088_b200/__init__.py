"""B200-native tree-verification step for EAGLE-3-style tree speculative
decoding: Python binding of the sm_100a C-ABI library (libtreeverify.so).

The entry points have the names of include/treeverify.h and only marshal
arguments; all arithmetic runs in the CUDA kernels.  PyTorch is used for
device memory and streams.  Importing this package does not load the shared
library; the first call does, and raises if it is missing.
"""
from .binding import (TreeVerifyError, load, tv_version, tv_launch_count, tree_build_mask, tree_verify_attn, tree_verify_attn_layers, tree_verify_attn_paged_layers,
                      tv_debug_attn_expire, tv_debug_attn_stream_only, TV_ATTN_STABLE_INPUTS, TV_ATTN_LAUNCH_PER_LAYER, tree_accept,
                      kv_commit, kv_commit_inplace, tree_verify_attn_paged, kv_commit_paged, tv_verify_step_host, tv_attn_workspace_bytes, tv_accept_workspace_bytes,
                      tv_step_staging_bytes, tv_debug_attn_simt, tree_accept_noalloc, tv_accept_noalloc_max_bytes, tree_node_scores, tree_merge_partials, tree_accept_sample, tv_sample_workspace_bytes, TV_ST_BAD_TREE, TV_ST_BAD_INDEX,
                      TV_ST_CAPACITY, TV_ST_TIMEOUT, TV_ST_PATHS_TRUNCATED, LIB_PATH, EXPORTS)
from .step import StepBuffers, verify_step

__all__ = [
    "TreeVerifyError", "load", "tv_version", "tv_launch_count", "tree_build_mask", "tree_verify_attn", "tree_verify_attn_layers", "tree_verify_attn_paged_layers", "tv_debug_attn_expire", "tv_debug_attn_stream_only", "TV_ATTN_STABLE_INPUTS", "TV_ATTN_LAUNCH_PER_LAYER", "tree_accept", "kv_commit", "kv_commit_inplace", "tree_verify_attn_paged", "kv_commit_paged",
    "tv_verify_step_host", "tv_attn_workspace_bytes", "tv_accept_workspace_bytes", "tv_step_staging_bytes",
    "tv_debug_attn_simt", "tree_accept_noalloc", "tv_accept_noalloc_max_bytes", "tree_node_scores", "tree_merge_partials", "tree_accept_sample", "tv_sample_workspace_bytes", "StepBuffers", "verify_step", "LIB_PATH", "EXPORTS",
    "TV_ST_BAD_TREE", "TV_ST_BAD_INDEX", "TV_ST_CAPACITY", "TV_ST_TIMEOUT", "TV_ST_PATHS_TRUNCATED",
]
