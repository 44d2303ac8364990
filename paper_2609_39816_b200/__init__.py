"""B200-native scheme GEMM (fast bilinear matrix multiplication at low precision).

Thin Python binding over the C-ABI library ``libfmm_b200.so`` (argument marshalling only;
every step of the path runs in the library's CUDA kernels).  There is no CPU fallback: importing
:mod:`paper_2609_39816_b200.binding` raises if the library has not been built.
"""
from .binding import (  # noqa: F401
    FmmError, Scheme, GemmDesc, SweepSummary, scheme_load, scheme_builtin, scheme_kron, scheme_permute_products, gauge_apply,
    scheme_gemm, scheme_gemm_workspace, scheme_gemm_workspace_layout, scheme_gemm_host, scheme_gemm_host_workspace, scheme_gemm_host_status, classical_gemm, classical_gemm_workspace, exact_gemm_f64,
    error_frobenius, error_frobenius_noalloc, error_frobenius_noalloc_max_elements, error_sweep, error_sweep_workspace, device_status, selftest_timeout, launch_count, lib_path,
    F32, BF16, E4M3, FLAG_REUSE_BHAT, FLAG_PRODUCTS_BF16, FLAG_SWEEP_SERIAL, FLAG_ROUND_PER_LEVEL, FLAG_SWEEP_UNFUSED, EXPORTED_SYMBOLS, profile_enable, profile_collect, PHASES,
    scheme_certificate, int8_quantize, hadamard_rotate, row_pow2_scale, row_unscale, scheme_joint_round_weights, int8_gemm_workspace, int8_gemm, int8_gemm_materialised_workspace, int8_gemm_materialised,
    scheme_certificate_corrected, int8_gemm_corrected_workspace, int8_gemm_corrected,
    int8_finegroup_control_workspace, int8_finegroup_control,
)
