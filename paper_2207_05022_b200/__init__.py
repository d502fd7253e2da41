"""B200-native shard decode + elastic transformer-layer execution (STI, arXiv 2207.05022).

The package is a thin ctypes binding over the C-ABI library built from `csrc/` (sm_100a CUDA).
Every step of the execution path runs in that library's kernels; Python only marshals arguments.
"""
from .binding import (  # noqa: F401
    STI_OK, STI_ATTN, STI_FFN, STI_F32, STI_BF16,
    StiError, StiModelDesc, StiShardCfg, StiShardBlob, StiStats,
    load_library, library_path,
    sti_ctx_create, sti_ctx_destroy, sti_ctx_set_layer_params, sti_plan_create, sti_plan_destroy,
    sti_shard_upload, sti_plan_finalize, sti_layer_forward, sti_model_forward, sti_model_forward_host,
    sti_sync, sti_shard_decode, sti_gemm_probe, sti_decode_rate_probe, sti_get_kernel_stamps, sti_plan_inject, sti_plan_retain, sti_shard_adopt, sti_plan_fill_stats, STI_INJECT_NONE, STI_INJECT_SLOW_COPY,
    STI_INJECT_PINNED_ALLOC_FAILURE, STAMP_KERNEL_NAMES, sti_plan_set_profiling, sti_plan_set_overlap, sti_get_stats, sti_plan_memory, sti_plan_check_guards,
    sti_ctx_launch_count, sti_host_retile, sti_strerror, sti_matrix_decode_noalloc, sti_plan_auto, sti_preload_after_run,
    sti_quantize_units, sti_quantize_units_by, sti_quantize_workspace_bytes, STI_QUANTIZE_SELECT, STI_QUANTIZE_SORT,
    Session,
)
