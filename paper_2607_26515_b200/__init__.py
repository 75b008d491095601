"""B200-native (sm_100a) Rollout-ResQ FP4 linear layer: Python binding of the C ABI in include/resq.h."""
from .binding import (  # noqa: F401
    OUT_BF16, OUT_F32, PATTERN_NAMES, S_2_4, S_BLOCK, S_CHAN50, S_DENSE, S_NONE, S_ROW50, ResqError,
    alloc_workspace, check, dequantize, last_error, lib, pack_weight, quantize_act, residual_mask,
    residual_mask_workspace_bytes, resq_linear, resq_workspace_bytes, w4a16_linear, w4a8_linear, w16a4_linear, swiglu_resq_linear, rmsnorm_resq_linear, rht_pack_weight, rht_resq_linear, keep_quarters, per_strip, kernel_launches, profile_enable,
    profile_read, KERNEL_KINDS, residual_mask_static, STATIC_SCRATCH_MAX_SCORES,
    debug_expire_next_wait, pack_weight_transposed, dgrad_linear, wgrad_linear, resq_linear_group, resq_group_workspace_bytes, MAX_GROUP,
)
