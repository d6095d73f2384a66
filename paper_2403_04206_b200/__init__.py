"""B200-native GRAWA / MGRAWA / LGRAWA averaging update.

The product is the CUDA library ``libgrawa.so`` (C ABI in ``include/grawa.h``); this package is
its thin ctypes binding.  Importing the package does not load the library; the first call does,
and fails loudly when the library cannot be built or loaded.  There is no CPU fallback.
"""
from .binding import (  # noqa: F401
    GrawaError,
    GRAWA_MAX_WORKERS,
    grawa_clear_plans,
    grawa_collect_kernel_times,
    grawa_debug_bounds_violations,
    grawa_get_option,
    grawa_grawa_step,
    grawa_last_cuda_error,
    grawa_last_step_status,
    grawa_launch_count,
    grawa_layer_norms,
    grawa_layer_sumsq,
    grawa_step_from_layer_sums,
    grawa_norm_ema,
    grawa_step_from_layer_norms,
    grawa_lgrawa_step,
    grawa_mgrawa_step,
    grawa_prox_step,
    grawa_selftest_bounded_wait,
    grawa_set_option,
    grawa_status_string,
    grawa_step_host,
    grawa_step_typed,
    grawa_sumsq_static,
    grawa_trace_read,
    grawa_version,
    grawa_workspace_bytes,
    library,
)
