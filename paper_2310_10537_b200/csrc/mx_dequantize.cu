// MX -> float conversion (Section 2 of arXiv 2310.10537): v_i = X * P_i, and
// every element of a block is NaN when the scale X is NaN.
//
// A pure stream bound by HBM bandwidth: bits/8 + 1/32 bytes read and 2 or 4
// bytes written per element.
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


// ---- conversion-free decode -----------------------------------------------------
// Element code e of the thread's packed words, moved to the top of a 32-bit word (sign at bit 31).
template <int BITS, int KWORDS>
__device__ __forceinline__ uint32_t code_at_top(const uint32_t (&w)[KWORDS], int e) {
  const int pos = BITS * e, wi = pos / 32, off = pos % 32;
  // (the shift runs on the multiply-add unit: the logic / shift pipe is this kernel's busiest)
  if (off + BITS <= 32) return off + BITS == 32 ? w[wi] : imad(w[wi], 1u << (32 - BITS - off), 0u);
  return __funnelshift_r(w[wi], w[(wi + 1) % KWORDS], off) << (32 - BITS);  // 6-bit code across two words
}

// Value of the code whose bits sit at the top of t, times fix = 2^(127 - bias) ... returned
// WITHOUT that factor: the caller multiplies by fix and by the block scale (both exact).
// The magnitude bits are dropped into an FP32 exponent/mantissa field: for normal codes that is
// the value / 2^(127 - bias), and for the format's subnormal codes it is an FP32 subnormal with
// the same meaning, which the multiply then normalises -- no special cases.  NaN / Inf codes of
// the FP8 formats are NOT handled here (the caller tests for them once per thread).
template <int FMT>
__device__ __forceinline__ float raw_value(uint32_t t) {
  if (FMT == MX_INT8) {
    const int n = (int)t >> 24;                                         // two's complement byte
    return __uint_as_float(0x4B400000u + (uint32_t)n) - 12582912.0f;    // exact int -> float
  }
  constexpr int W = FmtTraits<FMT>::bits;
  constexpr int MSHIFT = (FMT == MX_E4M3 || FMT == MX_E2M3) ? 20 : (FMT == MX_E2M1 ? 22 : 21);
  constexpr uint32_t MASK = ((1u << (W - 1)) - 1u) << MSHIFT;
  constexpr int SH = (32 - W) - MSHIFT;
  // the arithmetic shift drags copies of the sign along down to the magnitude field's top: one
  // mask keeps bit 31 and the magnitude
  return __uint_as_float((uint32_t)((int32_t)t >> SH) & (0x80000000u | MASK));
}
template <int FMT>
__device__ __forceinline__ float bias_fix() {  // 2^(127 - bias); INT8: 2^-6
  return FMT == MX_E4M3 ? 1.329227995784916e36f      // 2^120
       : FMT == MX_E5M2 ? 5.192296858534828e33f      // 2^112
       : FMT == MX_E3M2 ? 2.1267647932558654e37f     // 2^124
       : FMT == MX_INT8 ? 0.015625f
                        : 8.507059173023462e37f;     // 2^126 (E2M3, E2M1)
}

// A thread produces 64 bytes of output: a whole block as BF16 (32 elements) or half
// a block as FP32 (16 elements), written with two 256-bit stores.
template <int FMT, int DTYPE, int LAYOUT, bool ALIGNED32>
__global__ void __launch_bounds__(kDqThreads)
dequantize_kernel(const uint8_t* __restrict__ elems, const uint8_t* __restrict__ scales,
                  void* __restrict__ out, uint32_t n_units, uint32_t kblocks, FastDiv kb_div) {
  constexpr int bits = FmtTraits<FMT>::bits;
  constexpr int kElems = DTYPE == MX_BF16 ? 32 : 16;
  constexpr int kLanes = kBlock / kElems;
  constexpr int kInBytes = kElems * bits / 8;  // 32/24/16 or 16/12/8
  constexpr int kWords = kInBytes / 4;
  pdl_prologue();
  for (uint32_t unit = blockIdx.x * kDqThreads + threadIdx.x; unit < n_units;
       unit += gridDim.x * kDqThreads) {
    uint32_t w[kWords];
    const uint8_t* src = elems + (size_t)unit * kInBytes;
    if (kInBytes == 32) {
      if (ALIGNED32) {
        uint32_t t[8];
        ld_stream_32(src, t);
#pragma unroll
        for (int i = 0; i < 8; ++i) w[i % kWords] = t[i];
      } else {
        const uint4 a = ld_stream_16(src), b = ld_stream_16(src + 16);
        w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w;
        w[4 % kWords] = b.x; w[5 % kWords] = b.y; w[6 % kWords] = b.z; w[7 % kWords] = b.w;
      }
    } else if (kInBytes == 16) {
      const uint4 a = ld_stream_16(src);
      w[0] = a.x; w[1] = a.y; w[2 % kWords] = a.z; w[3 % kWords] = a.w;
    } else if (kInBytes == 8) {
      const uint2 a = __ldg(reinterpret_cast<const uint2*>(src));
      w[0] = a.x; w[1] = a.y;
    } else if (kInBytes == 24) {  // 8-byte aligned
#pragma unroll
      for (int i = 0; i < 3; ++i) {
        const uint2 a = __ldg(reinterpret_cast<const uint2*>(src) + i);
        w[(2 * i) % kWords] = a.x; w[(2 * i + 1) % kWords] = a.y;
      }
    } else {  // 12 bytes, 4-byte aligned
#pragma unroll
      for (int i = 0; i < 3; ++i) w[i % kWords] = __ldg(reinterpret_cast<const uint32_t*>(src) + i);
    }
    const uint32_t blk = unit / kLanes;
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
    // Special cases are rare and decided once per thread: a NaN scale, element codes for NaN / Inf
    // (FP8 formats only), and scales so small that results can be FP32 subnormals (which BF16
    // output would have to round).  Everything else takes the conversion-free path below.
    bool special = sb == 255 || sb < 24;
    if (FMT == MX_E4M3) {  // 0x7F / 0xFF: low seven bits all ones
#pragma unroll
      for (int i = 0; i < kWords; ++i) special |= (((w[i] & 0x7F7F7F7Fu) + 0x01010101u) & 0x80808080u) != 0;
    } else if (FMT == MX_E5M2) {  // exponent field 31
#pragma unroll
      for (int i = 0; i < kWords; ++i) special |= (((w[i] & 0x7C7C7C7Cu) + 0x04040404u) & 0x80808080u) != 0;
    }
    char* dst = reinterpret_cast<char*>(out) + (size_t)unit * 64;
    uint32_t o[16];
    if constexpr (FMT == MX_E2M1 && DTYPE == MX_BF16) {
      if (!special) {
        // 4-bit codes to BF16 without touching single elements: the eight magnitudes' BF16 bytes sit
        // in two 8-byte tables that a byte permute indexes with four code nibbles at once (the low
        // three bits of each; its fourth selector bit would replicate a sign, so it is masked off),
        // the signs come from a second permute in that sign-replicating mode, and X is one packed
        // BF16 multiply per pair (exact: the values have two significant bits and X is a power of
        // two whose products stay normal here, sb >= 24).
        //   magnitudes 0, 0.5, 1, 1.5, 2, 3, 4, 6 = 0x0000 3F00 3F80 3FC0 4000 4040 4080 40C0
        const uint32_t x2 = (sb << 7) * 0x00010001u;
#pragma unroll
        for (int i = 0; i < kWords; ++i) {
          const uint32_t n = w[i], mag = n & 0x77777777u, up = n << 4;
#pragma unroll
          for (int h = 0; h < 2; ++h) {  // codes 4 h .. 4 h + 3 of the word
            const uint32_t sel = h ? (mag >> 16) : (mag & 0xFFFFu);
            const uint32_t lo = __byte_perm(0xC0800000u, 0xC0804000u, sel);   // low bytes of the four values
            uint32_t hi = __byte_perm(0x3F3F3F00u, 0x40404040u, sel);         // high bytes
            // 0xFF where the code is negative: code 2 j + 1's sign is bit 7 of byte j of n, code 2 j's of n << 4
            const uint32_t neg = __byte_perm(n, up, h ? 0xBFAEu : 0x9D8Cu);
            hi |= neg & 0x80808080u;
            const uint32_t p0 = __byte_perm(lo, hi, 0x5140), p1 = __byte_perm(lo, hi, 0x7362);
            asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(o[4 * i + 2 * h]) : "r"(p0), "r"(x2));
            asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(o[4 * i + 2 * h + 1]) : "r"(p1), "r"(x2));
          }
        }
      }
    }
    if (FMT == MX_E2M1 && DTYPE == MX_BF16 && !special) {
      // (done above)
    } else if (!special) {
      const float fix = bias_fix<FMT>();
      uint32_t r[kElems];
#pragma unroll
      for (int e = 0; e < kElems; ++e)
        r[e] = __float_as_uint(raw_value<FMT>(code_at_top<bits, kWords>(w, e)) * fix * X);  // both products exact
      if (DTYPE == MX_F32) {
#pragma unroll
        for (int i = 0; i < 16; ++i) o[i] = r[i % kElems];
      } else {
        // at most 7 significant bits and no FP32 subnormals here: the upper half IS the BF16 value
#pragma unroll
        for (int i = 0; i < 16; ++i) o[i] = __byte_perm(r[(2 * i) % kElems], r[(2 * i + 1) % kElems], 0x7632);
      }
    } else {
      uint32_t r[kElems];
#pragma unroll
      for (int i = 0; i < kElems / 2; ++i) {
        uint32_t pair;  // code(2i) | code(2i+1) << 8   (4-bit: both in the low byte)
        if (bits == 8) {
          pair = (w[i / 2] >> (16 * (i & 1))) & 0xFFFFu;
        } else if (bits == 4) {
          pair = (w[i / 4] >> (8 * (i & 3))) & 0xFFu;
        } else {
          const int bit = 12 * i;  // two 6-bit codes at bit offset 12 i of the stream
          uint32_t q = w[bit / 32] >> (bit % 32);
          if (bit % 32 > 20) q |= w[(bit / 32 + 1) % kWords] << (32 - bit % 32);
          q &= 0xFFFu;
          pair = (q & 0x3Fu) | ((q & 0xFC0u) << 2);
        }
        float a, b;
        decode_pair<FMT>(pair, a, b);
        a *= X;  // exact unless it overflows to Inf
        b *= X;
        r[2 * i] = (a != a) ? 0x7FC00000u : __float_as_uint(a);  // canonical quiet NaN
        r[2 * i + 1] = (b != b) ? 0x7FC00000u : __float_as_uint(b);
      }
      if (DTYPE == MX_F32) {
#pragma unroll
        for (int i = 0; i < 16; ++i) o[i] = r[i % kElems];
      } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const float lo = __uint_as_float(r[(2 * i) % kElems]), hi = __uint_as_float(r[(2 * i + 1) % kElems]);
          uint32_t pk;
          asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(pk) : "f"(hi), "f"(lo));  // round to nearest even
          if (lo != lo) pk = (pk & 0xFFFF0000u) | 0x7FC0u;   // the packed conversion gives 0x7FFF for NaN
          if (hi != hi) pk = (pk & 0x0000FFFFu) | 0x7FC00000u;
          o[i] = pk;
        }
      }
    }
    if (ALIGNED32) {
      const uint32_t o0[8] = {o[0], o[1], o[2], o[3], o[4], o[5], o[6], o[7]};
      const uint32_t o1[8] = {o[8], o[9], o[10], o[11], o[12], o[13], o[14], o[15]};
      st_32(dst, o0);
      st_32(dst + 32, o1);
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j)
        reinterpret_cast<uint4*>(dst)[j] = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
    }
  }
}

// Axis lengths that are not a multiple of 32: the packed rows are padded to whole blocks, the
// output rows are not.  One thread per block, element by element, on the exact decode path.
template <int FMT, int DTYPE, int LAYOUT>
__global__ void __launch_bounds__(kDqThreads)
dequantize_tail_kernel(const uint8_t* __restrict__ elems, const uint8_t* __restrict__ scales,
                       void* __restrict__ out, uint32_t rows, uint32_t L, uint32_t kblocks, uint64_t total_blocks) {
  constexpr int bits = FmtTraits<FMT>::bits;
  constexpr int kWords = bits;  // 32-bit words of codes per block
  pdl_prologue();
  for (uint64_t b = (uint64_t)blockIdx.x * kDqThreads + threadIdx.x; b < total_blocks;
       b += (uint64_t)gridDim.x * kDqThreads) {
    const uint32_t row = (uint32_t)(b / kblocks), kb = (uint32_t)(b - (uint64_t)row * kblocks);
    const uint32_t* src = reinterpret_cast<const uint32_t*>(elems + (size_t)row * (kblocks * (kBlock * bits / 8)) +
                                                            (size_t)kb * (kBlock * bits / 8));
    uint32_t w[kWords];
#pragma unroll
    for (int i = 0; i < kWords; ++i) w[i] = __ldg(src + i);
    const uint32_t sb = __ldg(scales + scale_offset<LAYOUT>(row, kb, kblocks));
    const float X = __uint_as_float(sb == 0 ? 0x00400000u : (sb == 255 ? 0x7FC00000u : sb << 23));
#pragma unroll
    for (int i = 0; i < kBlock / 2; ++i) {
      uint32_t pair;  // code(2i) | code(2i+1) << 8   (4-bit: both in the low byte)
      if (bits == 8) {
        pair = (w[i / 2] >> (16 * (i & 1))) & 0xFFFFu;
      } else if (bits == 4) {
        pair = (w[i / 4] >> (8 * (i & 3))) & 0xFFu;
      } else {
        const int bit = 12 * i;
        uint32_t q = w[bit / 32] >> (bit % 32);
        if (bit % 32 > 20) q |= w[(bit / 32 + 1) % kWords] << (32 - bit % 32);
        q &= 0xFFFu;
        pair = (q & 0x3Fu) | ((q & 0xFC0u) << 2);
      }
      float v[2];
      decode_pair<FMT>(pair, v[0], v[1]);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const uint32_t k = kb * kBlock + 2 * i + h;
        if (k >= L) continue;
        const float r = v[h] * X;  // exact unless it overflows to Inf
        const size_t idx = (size_t)row * L + k;
        if (DTYPE == MX_F32) {
          reinterpret_cast<uint32_t*>(out)[idx] = (r != r) ? 0x7FC00000u : __float_as_uint(r);
        } else {
          uint32_t pk;
          asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(pk) : "f"(0.0f), "f"(r));  // round to nearest even
          reinterpret_cast<uint16_t*>(out)[idx] = (r != r) ? (uint16_t)0x7FC0u : (uint16_t)(pk & 0xFFFFu);
        }
      }
    }
  }
}

template <int FMT, int DTYPE, int LAYOUT>
static cudaError_t launch_dq(const DequantizeArgs& a) {
  if (a.L % kBlock != 0) {
    const uint32_t kb = (uint32_t)((a.L + kBlock - 1) / kBlock);
    const uint64_t total = (uint64_t)a.rows * kb;
    const uint64_t want = (total + kDqThreads - 1) / kDqThreads, cap = (uint64_t)a.sm_count * 64;
    return launch_pdl(dequantize_tail_kernel<FMT, DTYPE, LAYOUT>, dim3((uint32_t)(want < cap ? want : cap)),
                      dim3(kDqThreads), 0, a.stream, a.elems, a.scales, a.out, (uint32_t)a.rows, (uint32_t)a.L, kb,
                      total);
  }
  constexpr int kElems = DTYPE == MX_BF16 ? 32 : 16;
  const uint32_t n_units = (uint32_t)(a.rows * a.L / kElems);
  const uint32_t kblocks = (uint32_t)(a.L / kBlock);
  const FastDiv kd = make_fastdiv(kblocks);
  const bool al32 = (uintptr_t)a.out % 32 == 0 && (uintptr_t)a.elems % 32 == 0;
  auto kernel = al32 ? dequantize_kernel<FMT, DTYPE, LAYOUT, true> : dequantize_kernel<FMT, DTYPE, LAYOUT, false>;
  const uint32_t grid = (n_units + kDqThreads - 1) / kDqThreads;  // one CTA per 256 units, no loop
  return launch_pdl(kernel, dim3(grid), dim3(kDqThreads), 0, a.stream, a.elems, a.scales, a.out, n_units, kblocks, kd);
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
