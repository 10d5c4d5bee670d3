// Internal interface between the C ABI (mx_api.cu) and the kernel files.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "mx.h"

namespace mx {

struct QuantizeArgs {
  const void* in;
  uint8_t* elems;
  uint8_t* scales;
  int64_t outer, L, inner;  // input viewed as [outer, L, inner], blocks along L
  int64_t L_store;          // elements per stored row: L rounded up to whole blocks, or to 128 (zero codes)
  int64_t numel;
  int fmt, rounding, dtype, layout;
  int sm_count;
  cudaStream_t stream;
};
cudaError_t launch_quantize(const QuantizeArgs& a);

struct DualArgs {
  const void* in;
  uint8_t *elems_row, *scales_row;  // blocks along the contiguous axis: [R x C]
  uint8_t *elems_col, *scales_col;  // blocks along axis 0: [C x R]
  int64_t R, C;
  int fmt, rounding, dtype, layout;
  int sm_count;
  cudaStream_t stream;
};
// FP32 input, register kernel (mx_quantize_dual.cu).
cudaError_t launch_quantize_dual(const DualArgs& a);
// The same for BF16 input through TMA tiles in shared memory (mx_quantize_tile.cu).
cudaError_t launch_quantize_tile(const DualArgs& a);
// FP32 input, 6-bit codes, R and C multiples of 128, through the same kind of kernel.
cudaError_t launch_quantize_tile_f32(const DualArgs& a);
// The BF16 kernel's column pass alone (elems_row / scales_row unused): axis-0 quantize of a 2-D BF16
// tensor with 6- or 4-bit codes, R, C % 128 == 0.
cudaError_t launch_quantize_tile_cols(const DualArgs& a);
// Synchronises the stream, then reads and clears the tile kernels' status word (nonzero: a
// bounded device-side wait gave up).
cudaError_t quantize_tile_status(cudaStream_t stream, unsigned int* status);

struct DequantizeArgs {
  const uint8_t* elems;
  const uint8_t* scales;
  void* out;
  int64_t rows, L;
  int fmt, dtype, layout;
  int sm_count;
  cudaStream_t stream;
};
cudaError_t launch_dequantize(const DequantizeArgs& a);

// Activation x[N, H, W, C] quantized along C -> K-major operand [N Ho Wo x kh kw C] (see mx_im2col()).
struct Im2colArgs {
  const uint8_t* elems_in;
  const uint8_t* scales_in;
  uint8_t* elems_out;
  uint8_t* scales_out;  // swizzled
  int64_t N, H, W, C, Ho, Wo;
  int kh, kw, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w;
  int bits, layout_in;
  int sm_count;
  cudaStream_t stream;
};
cudaError_t launch_im2col(const Im2colArgs& a);

// Convolution without a materialized operand (see mx_conv2d()): x quantized along C (8-bit codes),
// filter w[Cout][kh kw C] quantized along its last axis (any block-scaled format, swizzled scales).
struct ConvArgs {
  const uint8_t* x_elems;
  const uint8_t* x_scales;
  const void* w_elems;
  const uint8_t* w_scales;
  void* y;  // FP32 or BF16 [N Ho Wo x Cout]
  int y_bf16;
  int64_t N, H, W, C, Ho, Wo, Cout;
  int kh, kw, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w;
  int fmt_x, fmt_w, x_layout;
  int sm_count;
  cudaStream_t stream;
};
// Returns MX_OK or a negative mx_status_t; fills *cuda_err on MX_ERR_CUDA.
int launch_conv(const ConvArgs& a, cudaError_t* cuda_err);

struct GemmArgs {
  const void* A;
  const uint8_t* sA;
  const void* B;
  const uint8_t* sB;
  void* C;      // FP32 [M x N], or BF16 when c_bf16 is nonzero
  int c_bf16;
  // When q_elems is set the epilogue quantizes C along N instead of storing it: packed codes
  // [batch*M x N] and swizzled scales (rows batch*M, N / 32 blocks); C is then unused.
  void* q_elems;
  uint8_t* q_scales;
  int q_fmt, q_round;
  // dense != 0: A and B are BF16 K-major matrices (dequantized MX tensors), sA / sB unused.
  int dense;
  int64_t batch;  // independent products; operands and C are the matrices stacked along rows
  int64_t M, N, K;
  int fmtA, fmtB;
  int force_bn;  // 0: let launch_gemm choose the tile width; 256 / 384: pin it (tuning and tests)
  int skinny_m;  // products with M <= skinny_m (at most 128) take the swapped-operand kernel
  int64_t wait_cycles;  // budget of a device-side wait in SM clock cycles; <= 0: the default (~1 s)
  int drop_fill;        // failure drill: the operand producer leaves out this pipeline fill; < 0: off
  int sm_count;
  cudaStream_t stream;
};
// Returns MX_OK or a negative mx_status_t; fills *cuda_err on MX_ERR_CUDA.
int launch_gemm(const GemmArgs& a, cudaError_t* cuda_err);
// Synchronises the stream, then reads and clears the per-device status word that a
// bounded device-side wait sets when it gives up (0 = every wait completed).
int gemm_status(cudaStream_t stream, unsigned int* status, cudaError_t* cuda_err);

}  // namespace mx
