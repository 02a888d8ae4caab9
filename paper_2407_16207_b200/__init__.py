"""B200 (sm_100a) verification kernels for Graph-structured Speculative Decoding.

Thin Python binding over the C-ABI library `libgsd.so` (see include/gsd.h): argument
marshalling only, every step of the path runs in the CUDA kernels.  There is no CPU
fallback: the calls raise if the library has not been built.
"""
from .binding import (GSD_ATTN_AUTO, GSD_ATTN_MMA, GSD_ATTN_SPLIT_BALANCED, GSD_ATTN_SPLIT_PER_SEQUENCE, GSD_ATTN_TCGEN05, GsdError, gsd_accept, gsd_accept_sampled, gsd_accept_sampled_workspace_bytes, gsd_accept_static, gsd_build_mask, gsd_unmerge_tree, gsd_draft_expand, gsd_commit_kv,
                      gsd_accept_workspace_bytes, gsd_verify_attn, gsd_verify_attn_num_splits,
                      gsd_verify_attn_workspace_bytes, gsd_verify_step_host,
                      gsd_verify_step_host_arena_bytes, gsd_version, gsd_debug_attn_wait, lib, library_path)

__all__ = ["GSD_ATTN_AUTO", "GSD_ATTN_MMA", "GSD_ATTN_SPLIT_BALANCED", "GSD_ATTN_SPLIT_PER_SEQUENCE", "GSD_ATTN_TCGEN05", "GsdError", "gsd_accept", "gsd_accept_sampled", "gsd_accept_sampled_workspace_bytes", "gsd_accept_static", "gsd_build_mask", "gsd_unmerge_tree", "gsd_draft_expand", "gsd_commit_kv",
           "gsd_accept_workspace_bytes", "gsd_verify_attn", "gsd_verify_attn_num_splits",
           "gsd_verify_attn_workspace_bytes", "gsd_verify_step_host",
           "gsd_verify_step_host_arena_bytes", "gsd_version", "gsd_debug_attn_wait", "lib", "library_path"]
