"""MX (Microscaling) quantize / dequantize / block-scaled GEMM for NVIDIA B200.

The package is a thin binding over ``libmx_b200.so`` (hand-written CUDA for
sm_100a behind the C ABI of ``include/mx.h``).  Importing it loads the library
and fails if it has not been built; nothing here computes on the CPU.
"""
from .binding import *  # noqa: F401,F403
from .binding import (EXPORTS, FORMATS, LIB_PATH, MxError, lib, mx_dequantize, mx_dequantize_host,
                      mx_dequantize_host_workspace_bytes, mx_elems_bytes, mx_fmt_bits, mx_gemm, mx_gemm_bf16, mx_gemm_ex, mx_gemm_batched, mx_gemm_quantize, mx_gemm_dense, mx_gemm_dense_workspace_bytes, mx_conv_geometry, mx_conv_out_hw, mx_im2col, mx_conv2d, mx_conv_t, mx_host_synchronize,
                      mx_gemm_host, mx_gemm_host_workspace_bytes, mx_quantize, mx_quantize_dual, mx_quantize_host, mx_quantize_host_static,
                      mx_quantize_host_workspace_bytes, mx_scale_offset, mx_scales_bytes)
