"""Group-sparse convolution for NVIDIA B200: thin ctypes binding over libsbnn.so.

Every function here only marshals arguments into the C interface declared in
include/sbnn.h; all arithmetic runs in the library's CUDA kernels.  There is
no CPU fallback: if the shared library is missing, importing the binding's
functions raises.
"""
from .binding import (  # noqa: F401
    SBNN_BF16_TC,
    SBNN_OUT_CM,
    SBNN_BF16_GATHER,
    SBNN_RELU,
    MobileNetV1,
    Packed,
    SbnnError,
    avgpool,
    conv1x1_gs,
    conv1x1_gs_cm,
    conv1x1_gs_tuned,
    conv3x3_dense,
    conv3x3_gs,
    conv3x3_gs_cm,
    dwconv3x3,
    dwconv3x3_cm,
    dwconv3x3_conv1x1_gs_cm,
    dwconv3x3_pattern,
    get_async_status,
    head_noalloc,
    lib,
    lib_path,
    load_packed,
    mobilenet_v1_layer_shape,
    pack_dw_pattern,
    pack_weights,
    prepare,
    selftest_fma_rate,
    debug_set_packed_device,
    debug_check_packed,
    debug_plan_conv3x3,
    debug_poke_device_index,
    selftest_wait_timeout,
    status_str,
    to_channel_major,
)
