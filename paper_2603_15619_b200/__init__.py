"""B200 (sm_100a) implementation of the Mixture-of-Depths Attention operator.

``binding`` exposes the C ABI of ``include/moda.h`` (hand-written CUDA kernels behind it);
``synthetic`` holds the seeded input recipes; ``flops`` the FLOP / byte accounting of the
reported metric.  The CUDA library is loaded on first use and there is no fallback path.
"""
from .autograd import moda_attention  # noqa: F401
from .stack import DepthStream  # noqa: F401
from .slots import SlotBuffer  # noqa: F401
from .binding import (  # noqa: F401
    MODA_BWD_ACCUMULATE_DEPTH,
    MODA_BWD_ALL_STAGES,
    MODA_BWD_DETERMINISTIC,
    MODA_BWD_STAGE_DKDV,
    MODA_BWD_STAGE_DQ,
    MODA_BWD_STAGE_ROWTERMS,
    ModaError,
    alloc_depth_cache,
    alloc_depth_cache_e4m3,
    depth_cache_window,
    moda_attn_bwd,
    moda_attn_bwd_e4m3,
    moda_attn_bwd_gqa,
    moda_attn_bwd_gqa_pm,
    moda_attn_bwd_gqa_stages,
    moda_attn_bwd_stages,
    moda_attn_bwd_static_scratch,
    moda_attn_decode,
    moda_attn_decode_paged,
    moda_attn_decode_varlen,
    moda_attn_fwd,
    moda_attn_fwd_append,
    moda_attn_fwd_e4m3,
    moda_attn_fwd_gqa,
    moda_attn_fwd_gqa_pm,
    moda_attn_fwd_prefill,
    moda_bwd_workspace_bytes,
    moda_bwd_workspace_bytes_gqa,
    moda_decode_workspace_bytes,
    moda_depth_cache_append,
    moda_depth_cache_append_e4m3,
    moda_depth_cache_append_pm,
    moda_depth_cache_e4m3_bytes,
    moda_depth_cache_bytes,
    moda_depth_cache_unpack,
    moda_depth_cache_unpack_pm,
    moda_kv_project_append,
    moda_kv_project_append_e4m3,
    moda_attn_fwd_append_e4m3,
    moda_depth_slot_mass,
    moda_last_status,
    moda_selftest_wait_timeout,
    moda_version,
)
