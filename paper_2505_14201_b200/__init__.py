"""FLASH-D attention forward for NVIDIA B200: thin Python binding over the
C-ABI CUDA library ``libflashd.so`` (declared in ``include/flashd.h``).

The binding only marshals arguments; every step of the computation runs in the
library's CUDA kernels.  There is no CPU path: a call fails loudly when the
library or a CUDA device is missing.
"""
from .binding import (  # noqa: F401
    FlashdError, lib, lib_path, status_string, version, launch_count,
    flashd_attn_fwd, flashd_attn_fwd_ex, flashd_attn_fwd_f32, flashd_attn_fwd_perkey, flashd_attn_fwd_fp8,
    flashd_splitk_workspace_bytes, flashd_splitk_num_splits, flashd_splitk_partial,
    flashd_splitk_combine, flashd_attn_fwd_splitk, flashd_attn_fwd_splitk_static, flashd_attn_fwd_host,
    flashd_gqa_num_splits, flashd_gqa_partial, flashd_attn_fwd_gqa, MAX_GROUP,
    flashd_attn_fwd_pwl, PWL_MAX_SEGMENTS, flashd_splitk_partial_fp8kv, flashd_attn_fwd_splitk_fp8kv,
    flashd_splitk_partial_paged, flashd_attn_fwd_splitk_paged, flashd_attn_fwd_gqa_paged,
    flashd_skip_stats, flashd_last_device_status, BF16, F32, MAX_SPLITS, STATIC_SCRATCH_BYTES, EXPORTED_SYMBOLS,
)
