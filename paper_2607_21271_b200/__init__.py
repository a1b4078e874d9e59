"""Flash EQ-Linear hot path for NVIDIA B200 (sm_100a): a C-ABI CUDA library plus this thin binding."""

from . import binding, parallel, workloads  # noqa: F401
from .binding import (  # noqa: F401
    EQL_FLAG_CORRELATION, EQL_FLAG_FORCE_SIMT, EQL_FLAG_FORCE_STREAMING, EQL_FLAG_CTA_PAIR, EQL_FLAG_NO_CTA_PAIR, EQL_FLAG_GELU, EQL_FLAG_DIHEDRAL, EQL_BF16, EQL_FP16, EQL_FP32, EqlError,
    eqlinear_bwd_data, eqlinear_bwd_data_host, eqlinear_bwd_weight, eqlinear_bwd_weight_host,
    eqlinear_bwd_weight_from_spectrum, eqlinear_bwd_weight_scratch_bytes, eqlinear_bwd_weight_static, eqlinear_count_macs, eqlinear_fwd, eqlinear_fwd_host, eqlinear_fwd_save_spectrum, eqlinear_spectrum_bytes, eqlinear_plan,
    eqlinear_plan_clear_device_status, eqlinear_plan_destroy, eqlinear_plan_device_status, eqlinear_plan_info, eqlinear_plan_launch_counts,
    eqlinear_plan_selftest_expired_wait, eqlinear_plan_set_weight, eqlinear_step_host,
    eqlinear_workspace_bytes, eqlinear_workspace_bytes_flags, load_library, status_string,
)
