"""B200-native (sm_100a) implementation of the USV sparsified attention hot path.

Thin Python binding over the C-ABI library ``libusv.so`` (see ``include/usv.h``): argument
marshalling only, every step of the path runs in the library's CUDA kernels.  PyTorch supplies
device memory and streams.
"""
from .binding import (  # noqa: F401
    USVError, lib, lib_path, block_scores, block_scores_noalloc, select_blocks, sparse_attn_fwd, token_merge,
    token_unmerge, MergePlan, workspace_status, sparse_attn_fallbacks, build_info, BLOCK, attn_entropy,
    allocate_sparsity, cube_order, permute_tokens, force_own_block, selftest_wait_timeout, kernel_launches, exclude_own_block, attn_combine, unmerge_map, sparse_attn_fwd_unmerge, merge_plan_cache, token_merge_apply,
)
