// MX -> float conversion (Section 2 of arXiv 2310.10537): v_i = X * P_i, and
// every element of a block is NaN when the scale X is NaN.
//
// A pure stream bound by HBM bandwidth: bits/8 + 1/32 bytes read and 2 or 4
// bytes written per element.  8 elements per thread, 4 lanes per MX block.
#include <cuda_fp16.h>

#include "mx_device.cuh"
#include "mx_launch.h"

namespace mx {

constexpr int kDqThreads = 256;

// Two codes -> two FP32 values (exact: every element value fits FP16).
// pair = code0 | code1 << 8  (FP4: code0 | code1 << 4 in the low byte).
template <int FMT>
__device__ __forceinline__ void decode_pair(uint32_t pair, float& a, float& b) {
  if (FMT == MX_INT8) {
    a = (float)(int8_t)(pair & 0xFF) * 0.015625f;
    b = (float)(int8_t)((pair >> 8) & 0xFF) * 0.015625f;
    return;
  }
  uint32_t h2;
  const uint16_t p = (uint16_t)pair;
  if (FMT == MX_E4M3) asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(p));
  else if (FMT == MX_E5M2) asm("cvt.rn.f16x2.e5m2x2 %0, %1;" : "=r"(h2) : "h"(p));
  else if (FMT == MX_E3M2) asm("cvt.rn.f16x2.e3m2x2 %0, %1;" : "=r"(h2) : "h"(p));
  else if (FMT == MX_E2M3) asm("cvt.rn.f16x2.e2m3x2 %0, %1;" : "=r"(h2) : "h"(p));
  else
    asm("{ .reg .b8 lo, hi; mov.b16 {lo, hi}, %1; cvt.rn.f16x2.e2m1x2 %0, lo; }"
        : "=r"(h2) : "h"(p));
  const __half2 h = *reinterpret_cast<const __half2*>(&h2);
  const float2 f = __half22float2(h);
  a = f.x;
  b = f.y;
}

template <int FMT, int DTYPE, int LAYOUT, bool ALIGNED32>
__global__ void __launch_bounds__(kDqThreads)
dequantize_kernel(const uint8_t* __restrict__ elems, const uint8_t* __restrict__ scales,
                  void* __restrict__ out, uint32_t n_chunks, uint32_t kblocks, FastDiv kb_div) {
  constexpr int bits = FmtTraits<FMT>::bits;
  for (uint32_t c = blockIdx.x * kDqThreads + threadIdx.x; c < n_chunks;
       c += gridDim.x * kDqThreads) {
    // 8 codes as four byte pairs
    uint32_t pair[4];
    if (bits == 8) {
      const uint2 w = __ldg(reinterpret_cast<const uint2*>(elems + (size_t)c * 8));
      pair[0] = w.x & 0xFFFF; pair[1] = w.x >> 16; pair[2] = w.y & 0xFFFF; pair[3] = w.y >> 16;
    } else if (bits == 4) {
      const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(elems + (size_t)c * 4));
#pragma unroll
      for (int i = 0; i < 4; ++i) pair[i] = (w >> (8 * i)) & 0xFF;
    } else {
      const uint16_t* p = reinterpret_cast<const uint16_t*>(elems + (size_t)c * 6);
      const uint64_t w = (uint64_t)__ldg(p) | ((uint64_t)__ldg(p + 1) << 16) | ((uint64_t)__ldg(p + 2) << 32);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t q = (uint32_t)(w >> (12 * i)) & 0xFFFu;  // two 6-bit codes
        pair[i] = (q & 0x3F) | ((q & 0xFC0) << 2);
      }
    }
    const uint32_t blk = c >> 2;
    size_t off;
    if (LAYOUT == MX_SCALES_LINEAR) {
      off = blk;
    } else {
      const uint32_t row = fastdiv(blk, kb_div);
      off = scale_offset<LAYOUT>(row, blk - row * kblocks, kblocks);
    }
    const uint32_t sb = __ldg(scales + off);
    // X = 2^(sb - 127); sb = 0 is the FP32 subnormal 2^-127, sb = 255 is NaN
    const float X = __uint_as_float(sb == 0 ? 0x00400000u : (sb == 255 ? 0x7FC00000u : sb << 23));
    uint32_t r[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float a, b;
      decode_pair<FMT>(pair[i], a, b);
      a *= X;  // exact unless it overflows to Inf
      b *= X;
      r[2 * i] = (a != a) ? 0x7FC00000u : __float_as_uint(a);
      r[2 * i + 1] = (b != b) ? 0x7FC00000u : __float_as_uint(b);
    }
    if (DTYPE == MX_F32) {
      if (ALIGNED32) {
        st_32(reinterpret_cast<char*>(out) + (size_t)c * 32, r);
      } else {
        uint4* o = reinterpret_cast<uint4*>(out) + (size_t)c * 2;
        o[0] = make_uint4(r[0], r[1], r[2], r[3]);
        o[1] = make_uint4(r[4], r[5], r[6], r[7]);
      }
    } else {
      uint32_t w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float lo = __uint_as_float(r[2 * i]), hi = __uint_as_float(r[2 * i + 1]);
        uint32_t pk;
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(pk) : "f"(hi), "f"(lo));  // round to nearest even
        if (lo != lo) pk = (pk & 0xFFFF0000u) | 0x7FC0u;
        if (hi != hi) pk = (pk & 0x0000FFFFu) | 0x7FC00000u;
        w[i] = pk;
      }
      reinterpret_cast<uint4*>(out)[c] = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
}

template <int FMT, int DTYPE, int LAYOUT>
static cudaError_t launch_dq(const DequantizeArgs& a) {
  const uint32_t n_chunks = (uint32_t)(a.rows * a.L / 8);
  const uint32_t kblocks = (uint32_t)(a.L / kBlock);
  uint32_t grid = (n_chunks + kDqThreads - 1) / kDqThreads;
  const uint32_t cap = (uint32_t)a.sm_count * 32;
  if (grid > cap) grid = cap;
  const FastDiv kd = make_fastdiv(kblocks);
  if (DTYPE == MX_F32 && (uintptr_t)a.out % 32 == 0)
    dequantize_kernel<FMT, DTYPE, LAYOUT, true><<<grid, kDqThreads, 0, a.stream>>>(
        a.elems, a.scales, a.out, n_chunks, kblocks, kd);
  else
    dequantize_kernel<FMT, DTYPE, LAYOUT, false><<<grid, kDqThreads, 0, a.stream>>>(
        a.elems, a.scales, a.out, n_chunks, kblocks, kd);
  return cudaGetLastError();
}

template <int FMT>
static cudaError_t dispatch_dq(const DequantizeArgs& a) {
  if (a.dtype == MX_BF16) {
    return a.layout == MX_SCALES_LINEAR ? launch_dq<FMT, MX_BF16, MX_SCALES_LINEAR>(a)
                                        : launch_dq<FMT, MX_BF16, MX_SCALES_SWIZZLED>(a);
  }
  return a.layout == MX_SCALES_LINEAR ? launch_dq<FMT, MX_F32, MX_SCALES_LINEAR>(a)
                                      : launch_dq<FMT, MX_F32, MX_SCALES_SWIZZLED>(a);
}

cudaError_t launch_dequantize(const DequantizeArgs& a) {
  switch (a.fmt) {
    case MX_E4M3: return dispatch_dq<MX_E4M3>(a);
    case MX_E5M2: return dispatch_dq<MX_E5M2>(a);
    case MX_E3M2: return dispatch_dq<MX_E3M2>(a);
    case MX_E2M3: return dispatch_dq<MX_E2M3>(a);
    case MX_E2M1: return dispatch_dq<MX_E2M1>(a);
    default: return dispatch_dq<MX_INT8>(a);
  }
}

}  // namespace mx
