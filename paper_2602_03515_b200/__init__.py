"""Basis-rotation optimizer step for B200: thin Python binding over the C-ABI library libbr.so.

Importing this package does not load the CUDA library; the first call that needs it does, and
fails loudly if it has not been built (there is no CPU fallback).
"""
from .binding import (  # noqa: F401
    BR_OK, BR_WARMUP, BR_WARN_RANK_DEFICIENT, BR_ERR_INVALID, BR_ERR_SHAPE, BR_ERR_DTYPE, BR_ERR_TAU,
    BR_ERR_OOM, BR_ERR_CUDA, BR_ERR_STATE, BR_ERR_TIMEOUT,
    BR_GEOM_NONE, BR_GEOM_UNILATERAL, BR_GEOM_BILATERAL, BR_SRC_FIRST, BR_SRC_SECOND,
    BR_F32, BR_BF16, BR_GEMM_FP32, BR_GEMM_BF16, BR_ACCUM_EVERY_STEP, BR_ACCUM_ON_REFRESH,
    BR_BUF_W, BR_BUF_M, BR_BUF_V2, BR_BUF_U, BR_BUF_V, BR_BUF_L, BR_BUF_R, BR_BUF_RING, BR_BUF_MROT, BR_BUF_CLIP,
    BrError, BrLayerDesc, BrHparams, BrCounters, load_library, library_path,
    br_state_bytes, br_create, br_step, br_set_lr, br_refresh_basis, br_sync_status,
    br_get_counters, br_get_basis_flags, br_set_counters, br_get_state, br_set_state, br_get_launch_stats,
    br_profile, br_get_profile, br_stage_aware_freq, br_effective_delay, br_lr_warmup_cosine, br_destroy, br_strerror, br_last_error, br_gemm_bf16, br_power_static,
    BR_INJECT_NONE, BR_INJECT_LAUNCH_FAILURE, br_debug_inject, br_debug_wait_timeout, BR_FLAG_DEBUG_CANARY, br_debug_check_canaries,
    BasisRotation,
)
