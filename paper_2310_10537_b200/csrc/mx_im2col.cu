// Convolution as a dot product (Section 4.1 of arXiv 2310.10537 counts convolution among the
// dot-product operations whose operands are MX tensors): the activation x[N, H, W, C] is quantized
// once, in blocks of 32 consecutive channels, and this kernel lays the codes and scale bytes out as
// the K-major operand A[M x K] of mx_gemm, M = N Ho Wo output pixels, K = kh kw C with the channel
// innermost.  Because C is a multiple of the block size no MX block straddles two filter taps, so
// every block of A is a copy of a block of x (or zero where the tap falls into the padding): the
// expansion moves bytes and never requantizes.
//
// HBM-bound gather: a thread moves 16 bytes of codes (consecutive threads: consecutive chunks of
// one output row, so a warp writes 512 contiguous bytes), the input is re-read kh kw times, mostly
// from L2.  A second kernel places the scale bytes, one 32-bit word of the swizzled layout (four
// K-blocks of one row) per thread.
#include "mx_device.cuh"
#include "mx_launch.h"

namespace mx {

namespace {

struct ConvGeom {
  uint32_t H, W, Ho, Wo, kw;
  int32_t stride_h, stride_w, pad_h, pad_w, dil_h, dil_w;
  FastDiv d_wo, d_howo, d_kw;
};

// Input pixel (row of the quantized activation) that tap `tap` of output pixel m reads, or -1.
__device__ __forceinline__ int64_t source_pixel(const ConvGeom& g, uint32_t m, uint32_t tap) {
  const uint32_t n = fastdiv(m, g.d_howo), r = m - n * (g.Ho * g.Wo);
  const uint32_t ho = fastdiv(r, g.d_wo), wo = r - ho * g.Wo;
  const uint32_t i = fastdiv(tap, g.d_kw), j = tap - i * g.kw;
  const int32_t hi = (int32_t)ho * g.stride_h - g.pad_h + (int32_t)i * g.dil_h;
  const int32_t wi = (int32_t)wo * g.stride_w - g.pad_w + (int32_t)j * g.dil_w;
  if (hi < 0 || hi >= (int32_t)g.H || wi < 0 || wi >= (int32_t)g.W) return -1;
  return ((int64_t)n * g.H + hi) * g.W + wi;
}

constexpr int kThreads = 256;

// One thread per chunk of the output codes: VEC = 32 bytes (a whole sector per request) when the
// pixel's codes and both tensors allow it, else 16.  chunks_per_pixel = C * bits / 8 / VEC.
template <int VEC>
__global__ void __launch_bounds__(kThreads)
im2col_codes_kernel(const uint8_t* __restrict__ in, uint8_t* __restrict__ out, ConvGeom g, uint32_t taps,
                    uint32_t chunks_per_pixel, FastDiv d_cpp, FastDiv d_taps, uint32_t total_chunks) {
  pdl_prologue();
  // (64-bit loop counter: the stride added to an index near 2^32 must not wrap)
  for (uint64_t it = (uint64_t)blockIdx.x * kThreads + threadIdx.x; it < total_chunks;
       it += (uint64_t)gridDim.x * kThreads) {
    const uint32_t idx = (uint32_t)it;  // = (m * taps + tap) * chunks_per_pixel + chunk
    const uint32_t mt = fastdiv(idx, d_cpp), chunk = idx - mt * chunks_per_pixel;
    const uint32_t m = fastdiv(mt, d_taps), tap = mt - m * taps;
    const int64_t px = source_pixel(g, m, tap);
    uint8_t* dst = out + (size_t)idx * VEC;
    if (VEC == 32) {
      uint32_t v[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
      if (px >= 0) ld_stream_32(in + ((size_t)px * chunks_per_pixel + chunk) * 32, v);
      st_32(dst, v);
    } else {
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (px >= 0) v = __ldg(reinterpret_cast<const uint4*>(in + ((size_t)px * chunks_per_pixel + chunk) * 16));
      *reinterpret_cast<uint4*>(dst) = v;
    }
  }
}

// One thread per 32-bit word of the swizzled output scale tensor, padding rows and K-blocks included
// (they are written as 0).  cb = C / 32 blocks per pixel.
template <int LAYOUT_IN>
__global__ void __launch_bounds__(kThreads)
im2col_scales_kernel(const uint8_t* __restrict__ in, uint32_t* __restrict__ out, ConvGeom g, uint32_t M,
                     uint32_t taps, uint32_t cb, FastDiv d_cb, uint32_t in_rows, uint32_t words_per_row,
                     FastDiv d_wpr, uint64_t total_words) {
  pdl_prologue();
  const uint32_t kblocks = taps * cb;
  for (uint64_t idx = (uint64_t)blockIdx.x * kThreads + threadIdx.x; idx < total_words;
       idx += (uint64_t)gridDim.x * kThreads) {
    // logical (row, word) of this thread; rows run to the padded count
    const uint32_t row = (uint32_t)(idx / words_per_row);
    const uint32_t wq = (uint32_t)(idx - (uint64_t)row * words_per_row);
    uint32_t word = 0;
    if (row < M) {
#pragma unroll
      for (uint32_t b = 0; b < 4; ++b) {
        const uint32_t kb = 4 * wq + b;
        if (kb < kblocks) {
          const uint32_t tap = fastdiv(kb, d_cb), c = kb - tap * cb;
          const int64_t px = source_pixel(g, row, tap);
          if (px >= 0) {
            const size_t off = LAYOUT_IN == MX_SCALES_LINEAR
                                   ? (size_t)px * cb + c
                                   : scale_offset<MX_SCALES_SWIZZLED>((uint32_t)px, c, cb);
            word |= (uint32_t)__ldg(in + off) << (8 * b);
          }
        }
      }
    }
    // swizzled position of (row, 4 wq .. 4 wq + 3): one aligned word
    out[scale_offset<MX_SCALES_SWIZZLED>(row, 4 * wq, kblocks) / 4] = word;
  }
}

}  // namespace

cudaError_t launch_im2col(const Im2colArgs& a) {
  ConvGeom g;
  g.H = (uint32_t)a.H; g.W = (uint32_t)a.W; g.Ho = (uint32_t)a.Ho; g.Wo = (uint32_t)a.Wo; g.kw = (uint32_t)a.kw;
  g.stride_h = a.stride_h; g.stride_w = a.stride_w; g.pad_h = a.pad_h; g.pad_w = a.pad_w;
  g.dil_h = a.dil_h; g.dil_w = a.dil_w;
  g.d_wo = make_fastdiv(g.Wo); g.d_howo = make_fastdiv(g.Ho * g.Wo); g.d_kw = make_fastdiv(g.kw);
  const uint32_t taps = (uint32_t)(a.kh * a.kw);
  const uint32_t M = (uint32_t)(a.N * a.Ho * a.Wo);
  const uint32_t pixel_bytes = (uint32_t)(a.C * a.bits / 8);
  const bool wide = pixel_bytes % 32 == 0 && (uintptr_t)a.elems_in % 32 == 0 && (uintptr_t)a.elems_out % 32 == 0;
  const uint32_t cpp = pixel_bytes / (wide ? 32 : 16);
  const uint64_t total_chunks = (uint64_t)M * taps * cpp;  // below 2^32: checked by the caller
  const uint32_t cap = (uint32_t)a.sm_count * 32u;
  uint64_t blocks = (total_chunks + kThreads - 1) / kThreads;
  const dim3 cgrid((uint32_t)(blocks < cap ? blocks : cap));
  cudaError_t e =
      wide ? launch_pdl(im2col_codes_kernel<32>, cgrid, dim3(kThreads), 0, a.stream, a.elems_in, a.elems_out, g,
                        taps, cpp, make_fastdiv(cpp), make_fastdiv(taps), (uint32_t)total_chunks)
           : launch_pdl(im2col_codes_kernel<16>, cgrid, dim3(kThreads), 0, a.stream, a.elems_in, a.elems_out, g,
                        taps, cpp, make_fastdiv(cpp), make_fastdiv(taps), (uint32_t)total_chunks);
  if (e != cudaSuccess) return e;
  const uint32_t cb = (uint32_t)(a.C / 32);
  const uint32_t words_per_row = (taps * cb + 3) / 4;
  const uint32_t rows_padded = (M + 127) / 128 * 128;
  const uint64_t total_words = (uint64_t)rows_padded * words_per_row;
  blocks = (total_words + kThreads - 1) / kThreads;
  const dim3 grid((uint32_t)(blocks < cap ? blocks : cap));
  if (a.layout_in == MX_SCALES_LINEAR)
    return launch_pdl(im2col_scales_kernel<MX_SCALES_LINEAR>, grid, dim3(kThreads), 0, a.stream, a.scales_in,
                      (uint32_t*)a.scales_out, g, M, taps, cb, make_fastdiv(cb), (uint32_t)(a.N * a.H * a.W),
                      words_per_row, make_fastdiv(words_per_row), total_words);
  return launch_pdl(im2col_scales_kernel<MX_SCALES_SWIZZLED>, grid, dim3(kThreads), 0, a.stream, a.scales_in,
                    (uint32_t*)a.scales_out, g, M, taps, cb, make_fastdiv(cb), (uint32_t)(a.N * a.H * a.W),
                    words_per_row, make_fastdiv(words_per_row), total_words);
}

}  // namespace mx
