"""Python binding of the B200 fused LM-head + Top-K distillation library (include/hass.h).

Argument marshalling only: every step of the path runs in the CUDA library. The functions
have the names of the C entry points without the ``hass_`` prefix. torch is used for device
memory and streams. If the shared library has not been built the import fails; there is no
fallback of any kind.
"""
from .binding import (  # noqa: F401
    HassError,
    HASS_BF16,
    HASS_FP32,
    K_MAX,
    check,
    hca_attention_bwd,
    hca_attention_bwd_workspace_bytes,
    hca_attention_fwd,
    hca_attention_workspace_bytes,
    HCA_MAX_DRAFTS,
    combined_distill_fwd_bwd,
    combined_distill_workspace_bytes,
    kernel_launch_count,
    lib,
    PROFILE_KINDS,
    profile_enable,
    profile_summary,
    selftest_wait_expiry,
    status_string,
    topk_distill_bwd,
    topk_distill_fwd,
    topk_distill_fwd_bwd,
    topk_distill_fwd_bwd_draft,
    topk_distill_fwd_bwd_host,
    topk_distill_fwd_draft,
    topk_distill_fwd_static,
    topk_distill_fwd_static_scratch_bytes,
    STATIC_SCRATCH_MAX_BYTES,
    topk_distill_host_workspace_bytes,
    topk_distill_workspace_bytes,
    version,
    variant_distill_fwd_bwd,
    LOSS_TOPK,
    LOSS_TOP_P,
    LOSS_NORMED_TOPK,
    LOSS_BIDIR_TOPK,
)
