"""Exact softmax attention forward/backward for B200 (sm_100a) behind a C ABI.

``inputs`` (seeded synthetic inputs) works without the compiled library; the
binding (``attn_fwd``, ``attn_bwd`` and friends) loads ``libattn_b200.so`` on first
call and raises if it is missing -- there is no CPU fallback.
"""
from . import inputs  # noqa: F401
from . import binding  # noqa: F401
from .binding import (  # noqa: F401
    ATTN_OK,
    ATTN_ALGO_AUTO, ATTN_ALGO_FUSED, ATTN_ALGO_MATERIALIZED, ATTN_ALGO_SIMT, ATTN_BF16, ATTN_F32,
    ATTN_MASK_BLOCK_SPARSE, ATTN_MASK_BLOCK_SPARSE_CAUSAL, ATTN_MASK_CAUSAL, ATTN_MASK_ELEMENT, ATTN_MASK_NONE, AttnError, Cfg, Mask, attn_bwd, attn_bwd_noalloc, attn_bwd_preprocess,
    attn_bwd_workspace_bytes, attn_cfg_onchip_elems, attn_fwd, attn_fwd_workspace_bytes, attn_io_bound_elems,
    attn_io_bound_sparse_elems, attn_io_replay, attn_mask_from_coo, attn_kernel_launches, attn_noalloc_scratch_bytes, attn_noalloc_status, attn_selftest_wait_timeout, attn_supported_cfgs, attn_timing_collect, attn_timing_enable,
    attn_workspace_status, status_str,
    attn_project, attn_weight_grad, attn_weights_bwd, attn_weights_bwd_workspace_bytes,
)
