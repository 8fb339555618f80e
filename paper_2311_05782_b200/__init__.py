"""B200-native fault-injected mixed-precision GEMM (MPGemmFI hot path).

Thin binding over the C ABI declared in include/mpgemmfi.h: the functions here
have the same names as the library's entry points and only marshal arguments.
All arithmetic runs in the CUDA kernels; there is no CPU fallback, and loading
fails loudly when the CUDA library is missing.
"""
from .binding import (  # noqa: F401
    FP16, BF16, TF32,
    SITE_A, SITE_B, SITE_ACC, SITE_OUT, SITE_TERM,
    DETECT_NONE, DETECT_BOUNDCHECK, DETECT_RANGE_MAX, DETECT_RANGE_FLIP, CORRECT, TERM_HMMA_STEP, OUTPUT_RANGE, TERM_IN_FORMAT,
    STATUS_SITE_SKIPPED, STATUS_WAIT_LIMIT, MAX_FAULTS, INLINE_FAULTS, HEADER_WORDS, STATIC_MAX_TRIALS,
    TILES_AUTO, TILES_SINGLE, TILES_PAIR, mpgemmfi_set_tile_policy,
    SPLIT_AUTO, SPLIT_OFF, SPLIT_ON, mpgemmfi_set_split_policy,
    SITE_DTYPE, SITE_LOG_DTYPE, RECORD_DTYPE, SUMMARY_DTYPE,
    MpgemmfiError, library_path, load_library, exported_symbols,
    mpgemmfi_gemm, mpgemmfi_campaign, mpgemmfi_campaign_static, mpgemmfi_kstep, mpgemmfi_flags_bytes,
    mpgemmfi_flags_bitmap_offset, mpgemmfi_campaign_workspace_bytes,
    mpgemmfi_validate_sites, mpgemmfi_strerror, mpgemmfi_last_cuda_error, mpgemmfi_version,
    gemm, campaign, split_flags, mpgemmfi_campaign_summary, campaign_summary,
    mpgemmfi_operand_exponents, mpgemmfi_gemm_ranged, mpgemmfi_gemm_addend,
    mpgemmfi_set_wait_limit_ms, mpgemmfi_debug_break_handover, mpgemmfi_debug_launch_slot,
    mpgemmfi_gemm_out16, OUT_FP32, OUT_FP16, OUT_BF16, mpgemmfi_debug_segments, mpgemmfi_null_launch,
)
from .sharding import campaign_sharded, shard_range  # noqa: F401,E402
