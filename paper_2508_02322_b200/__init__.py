"""B200 (sm_100a) implementation of the CAMERA micro-expert analysis hot path.

`binding` wraps the C ABI of libcamera_b200.so (include/camera.h); `workloads` draws the seeded
synthetic layers and calibration tokens the tests and the benchmark run on.
"""
from . import workloads  # noqa: F401
from .binding import (  # noqa: F401
    CameraError, Layer, alloc_workspace, camera_alloc_bits, camera_analyze_layer_host,
    camera_analyze_workspace_bytes, camera_read_status, camera_score_layer, camera_score_workspace_bytes, camera_score_workspace_bytes_single_pass,
    camera_select_prune, camera_select_all, camera_select_workspace_bytes, camera_sub_index, camera_compact_weights,
    expert_offsets_tensor, camera_layer_forward, camera_score_forward_layer, camera_mask_down_columns, camera_pruned_output, camera_forward_workspace_bytes, camera_output_error, camera_residual_norm,
    camera_set_wait_limit_ns, camera_get_wait_limit_ns, camera_wait_probe, camera_select_prune_static,
    camera_layer_prepare, camera_layer_release, lib)
