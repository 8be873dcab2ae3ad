"""Backpropagation with pooling-compressed activations: B200 (sm_100a) hot path.

`api` binds the C-ABI CUDA library (libac.so, built in-tree from csrc/);
`synth` draws the seeded synthetic inputs used by the tests and the benchmark.
"""
from . import synth  # noqa: F401
from .api import (  # noqa: F401
    AcError, ConvDesc, ac_backward_step_host, ac_compress, ac_compress_relu_mask, ac_compress_relu_mask_y, ac_relu_mask_backward, ac_accumulate_workspace_bytes,
    ac_conv2d_wgrad_compressed_accumulate,
    ac_conv2d_wgrad_compressed,
    ac_conv2d_wgrad_compressed_static, ac_collapsed_workspace_bytes,
    ac_conv2d_wgrad_compressed_collapsed,
    ac_host_step_arena_bytes, ac_workspace_bytes_rect, ac_compress_rect, ac_conv2d_wgrad_compressed_rect,
    ac_selftest_bounded_wait, ac_set_kernel_timing_events, ac_set_sm_budget, ac_get_sm_budget, ac_wgrad_plan_info, ac_workspace_bytes, ac_workspace_bytes_min, ac_workspace_status, status_string,
)
