"""B200-native forward 2-D convolution (the operation optimised in arXiv 1705.10591).

The product is the C-ABI library ``libconv2d_b200.so`` declared in
``include/conv2d_b200.h``.  This package is its thin Python binding: argument
marshalling only -- every step of the computation runs in the CUDA kernels.
PyTorch is used by callers for device memory and streams, never for arithmetic.
"""
from .binding import (  # noqa: F401
    ALGO_16BIT, ALGO_AUTO, ALGO_FFMA, ALGO_TF32, FLAG_WEIGHTS_PACKED, OPERAND_BF16, OPERAND_FP16, Conv2dError,
    conv2d_fwd_general, conv2d_fwd_general_16bit, conv2d_fwd_general_noalloc, conv2d_fwd_general_padded,
    conv2d_fwd_general_strided, conv2d_fwd_host, conv2d_fwd_padded_workspace_size, conv2d_fwd_strided_workspace_size,
    conv2d_fwd_plan_describe, conv2d_fwd_single_channel, conv2d_fwd_workspace_size,
    conv2d_get_status, conv2d_launch_count, conv2d_status_string, library_path, load_library,
)
