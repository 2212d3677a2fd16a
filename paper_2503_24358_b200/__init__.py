"""SQuat KV-cache write path for NVIDIA B200 (sm_100a).

The product is the C-ABI shared library `libsquat.so` (declared in include/squat.h, built from
csrc/ by build.py).  This package is its thin Python binding: same names, argument marshalling
only, torch used for device memory and streams.
"""
from .binding import (  # noqa: F401
    EXPORTED_SYMBOLS, FLAG_BOUNDS, FLAG_DEVICE_TIMEOUT, FLAG_NO_CONVERGE, FLAG_NONFINITE, FLAG_ZERO_RANGE, LIB_PATH, SQUAT_BF16, SQUAT_F32,
    SQUAT_KEYS, SQUAT_VALUES, SquatError, Subspace, squat_build_subspace, squat_dequantize,
    squat_get_device_status, squat_gram_static, squat_kernel_launch_count, squat_quantize_keys, squat_quantize_values,
    squat_subspace_eig_sweeps, squat_subspace_export, squat_subspace_import, squat_write_path_host, squat_write_path_workspace_bytes,
    squat_decode_attention, squat_decode_attention_workspace_bytes, squat_decode_attention_pre_rope, squat_rope_table,
    squat_build_subspace_from_gram, squat_build_subspace_power, squat_build_subspace_power_from_gram, squat_build_subspace_sharded, token_shard, squat_fp32_peak_probe, squat_append_window_host, squat_subspace_select_key_kernel, squat_checked_selftest,
)
