"""B200-native MXAttention hot path: UOS-scaled MXFP4 quantization and the PNQ attention forward.

The compute lives in ``libmxattn.so`` (hand-written sm_100a CUDA behind a C ABI, declared in
``include/mxattn.h``).  This package is only the argument-marshalling binding; it has no CPU
fallback and raises if the library is missing.
"""
from .binding import (  # noqa: F401
    FLAG_HADAMARD, FLAG_OUT_FP32, FLAG_PNQ, FLAG_UOS, LAYOUT_CANONICAL, LAYOUT_TILE, MODE_HADAMARD, MODE_OCP, MODE_UOS,
    MxAttnError, device_status, forward, forward_bf16, forward_bf16_workspace_bytes, forward_cycle_profile, forward_cycle_profile_bytes, forward_debug_dump, forward_debug_dump_bytes, forward_host, forward_host_arena_bytes, forward_nvfp4, forward_nvfp4_workspace_bytes, forward_prequantized,
    forward_static, forward_workspace_bytes, forward_ws, last_launch_count, lib, lib_path, probe_fp4_gemm, quantize_mxfp4,
    quantize_mxfp4_batched, quantize_mxfp4_qmax, quantize_nvfp4, quantizer_status, tensor_amax, rowsum_diagnostic, selftest_bounded_wait, selftest_pair_abandon, set_workspace, strerror,
)
