"""B200-native EntropyInfer prefill path: thin Python binding over libentropyinfer (C ABI).

The binding only marshals arguments; every stage runs in the library's CUDA kernels.
PyTorch is used by callers for device memory and streams, not by this package's math.
"""
from .binding import (  # noqa: F401
    EiError,
    EiParams,
    EiCompressParams,
    compress_params,
    latent_compress,
    latent_compress_workspace_bytes,
    Plan,
    ITEM,
    STATUS,
    FLAG_ATTN_P_VIA_SMEM,
    FLAG_ATTN_SINGLE_TILE,
    FLAG_ATTN_PAIR_8WARP,
    FLAG_GROUP_SHARED,
    FLAG_PLAN_STAGED,
    FLAG_PLAN_FUSED,
    FLAG_ATTN_PERSISTENT,
    FLAG_ATTN_PER_CTA,
    FLAG_ATTN_NO_SKIP,
    FLAG_ATTN_SKIP_ZERO_PV,
    FLAG_ATTN_QUAD,
    FLAG_ATTN_SPLIT,
    FLAG_ATTN_TRI,
    FLAG_HEAD_SHARD,
    ROPE_NO_POOL,
    entropy_noalloc,
    lib,
    NOALLOC_SCRATCH_BYTES,
    load_library,
    params_default,
    status_string,
    version,
)
