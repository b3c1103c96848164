"""B200-native fused AdamS N:M optimizer step (CAST, arxiv 2509.25996).

The product is the C-ABI library built from csrc/ (see include/cast_adams.h);
`binding` mirrors its entry points for Python callers and `workloads` draws the
seeded synthetic inputs.  There is no CPU or PyTorch fallback.
"""
from . import binding, workloads  # noqa: F401
from .binding import (  # noqa: F401
    CastError, check,
    cast_adams_step, cast_adams_step_ex, cast_plan_step_stats, cast_scale_adam_step, cast_plan_scale_adam_step, cast_plan_create, cast_plan_create_ex, cast_plan_step, cast_plan_destroy, cast_plan_report_staging_failure,
    cast_host_ctx_create, cast_host_step, cast_host_ctx_sync, cast_host_ctx_destroy,
    cast_host_step_static, cast_kd_loss, cast_prune_fold, cast_plan_prune_fold, cast_mask_stats, cast_plan_mask_stats,
    cast_probe_launch, cast_probe_stream, cast_bulk_timeout_count,
    cast_strerror, cast_last_cuda_error, cast_kernel_launch_count,
)
