"""B200-native dual-precision (fast / full mode) linear layers over nested FP8 + residual planes.

The computation lives in ``libdps.so`` (hand-written CUDA for sm_100a behind the C ABI declared
in ``include/dps.h``); ``binding`` exposes the same calls to Python and ``workloads`` draws the
seeded synthetic inputs.
"""
from . import workloads  # noqa: F401
from .binding import (  # noqa: F401
    DPS_ENC_AUTO, DPS_ENC_AUTO_RN, DPS_ENC_E4M3, DPS_ENC_E4M3_RN, DPS_ENC_E5M2, DPS_ENC_E5M2_RN, DPS_MODE_FAST, DPS_MODE_FULL, DPS_OK, DpsError, dps_backup_residual, dps_debug_wait_timeout,
    dps_launch_count, dps_linear, dps_linear_fp8act, dps_moe_linear, dps_moe_linear_static, dps_moe_workspace_bytes,
    dps_quantize_activations, dps_reconstruct, dps_restore_residual, dps_split_weights, dps_stream_status, dps_version,
    library, status_string)
