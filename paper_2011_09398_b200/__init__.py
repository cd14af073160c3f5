"""B200 (sm_100a) binarized 2-D convolution: Python binding of the C-ABI CUDA library.

The functions here only marshal arguments (device pointers of torch tensors, the current
CUDA stream) into ``liblce_b200.so``; every step of the path runs in that library's
kernels.  There is no CPU fallback: without the built library or without a CUDA device
the calls raise.
"""
from .binding import (  # noqa: F401
    ACT_NONE, ACT_RELU, KERNEL_AUTO, KERNEL_DIRECT, KERNEL_TENSOR, KERNEL_TILED, OUT_BITPACKED, OUT_FLOAT32, OUT_INT32,
    PAD_SAME_ONE, PAD_SAME_ZERO, PAD_VALID, LceError, BConv2dDesc,
    lce_add_f32, lce_bconv2d, lce_bconv2d_plan, lce_bconv2d_plan_create, lce_plan_run, lce_plan_destroy, BConv2dPlan, lce_bconv2d_f32, lce_bconv2d_fused, lce_bconv2d_host, lce_bconv2d_host_async, lce_bconv2d_host_noalloc, lce_bconv2d_host_noalloc_max_bytes, lce_bconv2d_pack_weights, lce_bconv2d_packed_weights_bytes, lce_bconv2d_host_workspace_bytes, lce_bconv2d_out_shape,
    lce_bitpack, lce_bmaxpool, lce_device_status, lce_device_status_reset, lce_device_wait_probe, lce_status_string, lce_unpack, lce_version, library,
    make_desc, pack_weights,
)
