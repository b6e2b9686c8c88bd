"""B200 (sm_100a) forward pass of LASER's Segmented Target Attention + Global Stacked Target Attention.

The product is the C-ABI CUDA library `liblaser.so` (sources under csrc/, declarations in include/laser.h).
This package is its thin Python binding: argument marshalling of torch device tensors into the C calls.
Importing the package does not load the library; the first call does, and fails loudly if it is missing.
"""
from .binding import (  # noqa: F401
    LaserConfig,
    LaserError,
    DeviceBatch,
    PATH_AUTO, PATH_SIMT, PATH_TENSOR, PATH_STREAM,
    DTYPE_F32, DTYPE_BF16,
    load_library,
    library_path,
    make_config,
    laser_workspace_bytes,
    laser_workspace_regions,
    laser_selftest_wait_timeout,
    laser_host_transfer_bytes,
    laser_host_workspace_bytes,
    laser_sta_forward,
    laser_sta_forward_static,
    laser_gsta_forward,
    laser_fusion_forward,
    laser_sta_softmax_workspace_bytes,
    laser_sta_softmax_forward,
    laser_backward_workspace_bytes,
    laser_backward,
    laser_ffn_workspace_bytes,
    laser_ffn_forward,
    laser_forward_ffn,
    LaserFfnParams,
    laser_forward,
    laser_forward_packed,
    laser_forward_host,
    laser_check_status,
    laser_last_launch_count,
    laser_profile_enable,
    laser_profile_read,
    laser_status_string,
)
from .sharding import user_shard, shard_batch_arrays  # noqa: F401
