"""B200-native fused BF16 attention forward / backward with the GProj correction.

Public calls mirror the C ABI of ``include/gproj_attn.h``; they raise if the CUDA
library has not been built or the device is not sm_100a (there is no CPU path).
"""
from .binding import (  # noqa: F401
    FLAG_NO_K_CORRECTION,
    FLAG_NO_Q_CORRECTION,
    FLAG_ONLY_DKV_PASS,
    FLAG_ONLY_DQ_PASS,
    FWD_FLAG_FMA_SOFTMAX,
    GprojError,
    VarlenPlan,
    gproj_attn_bwd,
    gproj_attn_bwd_rect,
    gproj_attn_bwd_static_scratch,
    gproj_attn_bwd_varlen,
    gproj_attn_bwd_varlen_qk,
    gproj_attn_bwd_workspace_bytes,
    gproj_attn_fwd,
    gproj_attn_fwd_bwd_host,
    gproj_attn_fwd_rect,
    gproj_attn_host_staging_bytes,
    gproj_fp32_attn_bwd,
    gproj_fp32_attn_fwd,
    gproj_key_smooth,
    gproj_attn_fwd_varlen,
    gproj_attn_fwd_varlen_qk,
    gproj_last_device_status,
    gproj_last_launch_count,
    gproj_selftest_wait_timeout,
    status_string,
)
