// Device-side building blocks shared by the quantize / dequantize kernels:
// format traits, the narrow hardware casts of sm_100a, 128/256-bit global
// accesses and the per-block scale arithmetic of Algorithm 1 (Section 3 of
// arXiv 2310.10537).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "mx.h"

namespace mx {

constexpr int kBlock = 32;  // MX block size k (Table 1)

// Table 1 element formats: width of a code and emax_elem of Algorithm 1.
template <int FMT> struct FmtTraits;
template <> struct FmtTraits<MX_E4M3> { static constexpr int bits = 8, emax = 8; };
template <> struct FmtTraits<MX_E5M2> { static constexpr int bits = 8, emax = 15; };
template <> struct FmtTraits<MX_E3M2> { static constexpr int bits = 6, emax = 4; };
template <> struct FmtTraits<MX_E2M3> { static constexpr int bits = 6, emax = 2; };
template <> struct FmtTraits<MX_E2M1> { static constexpr int bits = 4, emax = 2; };
template <> struct FmtTraits<MX_INT8> { static constexpr int bits = 8, emax = 0; };

// Division by a run-time constant (32-bit dividend below 2^31) as multiply-high
// + shift; used to turn a flat block index into (row, kblock).
struct FastDiv {
  uint32_t d, mul, shift;
};
inline FastDiv make_fastdiv(uint32_t d) {
  FastDiv f;
  f.d = d;
  if (d == 1) { f.mul = 0; f.shift = 0; return f; }
  uint32_t s = 0;
  while ((1ull << s) < d) ++s;  // s = ceil(log2 d)
  f.shift = s;
  f.mul = (uint32_t)((((1ull << s) - d) << 32) / d + 1);
  return f;
}
__device__ __forceinline__ uint32_t fastdiv(uint32_t n, const FastDiv& f) {
  if (f.d == 1) return n;
  uint32_t t = __umulhi(n, f.mul);
  return (uint32_t)(((uint64_t)t + n) >> f.shift);
}

// Byte offset of the scale of (row, kb): see mx_scale_offset() in mx.h.
template <int LAYOUT>
__device__ __forceinline__ size_t scale_offset(uint32_t row, uint32_t kb, uint32_t kblocks) {
  if (LAYOUT == MX_SCALES_LINEAR) return (size_t)row * kblocks + kb;
  const uint32_t kchunks = (kblocks + 3) >> 2;
  const size_t chunk = (size_t)(row >> 7) * kchunks + (kb >> 2);
  return chunk * 512 + (row & 31) * 16 + ((row >> 5) & 3) * 4 + (kb & 3);
}

// ---- arithmetic primitives -------------------------------------------------

// a * b with subnormal inputs and results flushed to signed zero: applied to
// V_i this is exactly the "FP32 subnormal inputs give P_i = 0" rule.
__device__ __forceinline__ float mul_ftz(float a, float b) {
  float d;
  asm("mul.ftz.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
  return d;
}

// max(|a|, |b|) up to sign, NaN if either is NaN (the sign of the result is
// meaningless; callers only use the magnitude bits).
__device__ __forceinline__ float absmax_nan(float a, float b) {
  float d;
  asm("max.NaN.xorsign.abs.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
  return d;
}

// The same on two packed BF16 values per operand (the result's halves carry arbitrary signs).
__device__ __forceinline__ uint32_t absmax_nan_bf16x2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("max.NaN.xorsign.abs.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
// A float whose magnitude bits are the larger magnitude of the two BF16 halves of m.
__device__ __forceinline__ float bf16x2_halves_max(uint32_t m) {
  const uint32_t lo = (m << 16) & 0x7FFF0000u, hi = m & 0x7FFF0000u;
  return __uint_as_float(lo > hi ? lo : hi);  // magnitudes order like unsigned integers; NaN stays on top
}

// min(|x|, bound) with the sign of x (bound > 0): one instruction.
__device__ __forceinline__ float clamp_abs(float x, float bound) {
  float d;
  asm("min.xorsign.abs.f32 %0, %1, %2;" : "=f"(d) : "f"(x), "f"(bound));
  return d;
}

// Per-block scalars derived from the block maximum.
struct BlockScale {
  uint32_t byte;  // E8M0 scale byte: 0xFF for a block with Inf/NaN
  float m1, m2;   // V * m1 * m2 = V / X  (INT8: 64 * V / X); powers of two
  bool finite;
};

// amax: any float whose magnitude bits are those of max|V_i| (NaN if the block
// holds a NaN).  shared_exp = floor(log2 amax) - emax_elem, clamped at -127;
// a zero or all-subnormal block gets byte 0.
template <int FMT>
__device__ __forceinline__ BlockScale block_scale(float amax) {
  const uint32_t e = (__float_as_uint(amax) >> 23) & 0xFFu;  // biased exponent of amax
  BlockScale s;
  s.finite = (e != 0xFFu);
  const int emax = FmtTraits<FMT>::emax;
  const uint32_t b = e > (uint32_t)emax ? e - (uint32_t)emax : 0u;  // shared_exp + 127
  s.byte = s.finite ? b : 0xFFu;
  if (FMT == MX_INT8) {
    // 64 / X = 2^(133 - b) does not fit a float for small b: split it in two.
    const bool low = b < 128u;
    s.m1 = __uint_as_float((low ? 196u - b : 260u - b) << 23);  // 2^(69-b) or 2^(133-b)
    s.m2 = low ? 18446744073709551616.0f : 1.0f;                // 2^64 or 1
  } else {
    s.m1 = __uint_as_float((254u - b) << 23);  // 1 / X = 2^(127 - b), b <= 252 here
    s.m2 = 1.0f;
  }
  return s;
}

// Round (lo, hi) to the element grid with saturation; ROUND selects ties to
// even (the hardware cast) or ties away from zero.  Ties away is the same cast
// applied to the value with its last mantissa bit set: every tie of these grids
// has that bit clear, so a tie moves just past the half-way point and nothing
// else crosses one.
// Result: code(lo) | code(hi) << 8   (FP4: code(lo) | code(hi) << 4).
// CLAMP (INT8 only): false when the caller knows that no element of the block reaches 127.5 in
// magnitude after scaling (the saturation then has nothing to do).
template <int FMT, int ROUND, bool CLAMP = true>
__device__ __forceinline__ uint32_t cast_pair(float lo, float hi) {
  if (ROUND == MX_RHAZ) {
    lo = __uint_as_float(__float_as_uint(lo) | 1u);
    hi = __uint_as_float(__float_as_uint(hi) | 1u);
  }
  uint16_t p;
  if (FMT == MX_E4M3) {
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(p) : "f"(hi), "f"(lo));
  } else if (FMT == MX_E5M2) {
    asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(p) : "f"(hi), "f"(lo));
  } else if (FMT == MX_E3M2) {
    asm("cvt.rn.satfinite.e3m2x2.f32 %0, %1, %2;" : "=h"(p) : "f"(hi), "f"(lo));
  } else if (FMT == MX_E2M3) {
    asm("cvt.rn.satfinite.e2m3x2.f32 %0, %1, %2;" : "=h"(p) : "f"(hi), "f"(lo));
  } else if (FMT == MX_E2M1) {
    asm("{ .reg .b8 t; cvt.rn.satfinite.e2m1x2.f32 t, %1, %2; mov.b16 %0, {t, 0}; }"
        : "=h"(p) : "f"(hi), "f"(lo));
  } else {  // INT8: value n/64, inputs already multiplied by 64; saturate at +-127
    // x + 1.5 * 2^23 rounds x to an integer (nearest even) in the low mantissa bits, as two's
    // complement for negative x: no float-to-int conversion needed.
    const float a = (CLAMP ? clamp_abs(lo, 127.0f) : lo) + 12582912.0f;
    const float b = (CLAMP ? clamp_abs(hi, 127.0f) : hi) + 12582912.0f;
    p = (uint16_t)__byte_perm(__float_as_uint(a), __float_as_uint(b), 0x0040);  // low bytes of a and b
  }
  return p;
}

// a * b + c on the integer multiply-add unit (written as PTX so that it is not turned back into
// shifts and logic operations).
__device__ __forceinline__ uint32_t imad(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

// Packs the four code pairs of 8 consecutive elements (cast_pair results) into the block's
// little-endian bit stream: 8-bit formats lo = codes 0..3, hi = codes 4..7; 6-bit formats lo =
// bits 0..31, hi = bits 32..47; 4-bit format lo = all 32 bits.
template <int FMT>
__device__ __forceinline__ void pack8(const uint32_t (&p)[4], uint32_t& lo, uint32_t& hi) {
  constexpr int bits = FmtTraits<FMT>::bits;
  if (bits == 8) {
    lo = __byte_perm(p[0], p[1], 0x5410);
    hi = __byte_perm(p[2], p[3], 0x5410);
  } else if (bits == 4) {
    lo = imad(p[3], 1u << 24, imad(p[2], 1u << 16, imad(p[1], 1u << 8, p[0])));  // disjoint bytes: sums are ors
    hi = 0;
  } else {
    // Fields that do not overlap are joined by multiply-add instead of shift + or: the integer
    // multiply-add issues on the FMA pipe, which this kernel leaves idle, while the logic / shift
    // pipe is its busiest unit.  p = c0 + 256 c1 (codes below 64)  ->  q = c0 + 64 c1 = p - 192 (p >> 8).
    uint32_t q[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) q[i] = imad(p[i] >> 8, 0xFFFFFF40u, p[i]);  // 2 codes -> 12 bits
    lo = imad(q[2], 1u << 24, imad(q[1], 1u << 12, q[0]));
    hi = imad(q[3], 16u, q[2] >> 8);
  }
}

// Convert 8 consecutive elements of one block (output as pack8).
template <int FMT, int ROUND, bool CLAMP = true>
__device__ __forceinline__ void cast8(const float (&v)[8], const BlockScale& s, uint32_t& lo,
                                      uint32_t& hi) {
  uint32_t p[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float a = mul_ftz(v[2 * i], s.m1), b = mul_ftz(v[2 * i + 1], s.m1);
    if (FMT == MX_INT8) { a *= s.m2; b *= s.m2; }
    p[i] = cast_pair<FMT, ROUND, CLAMP>(a, b);
  }
  pack8<FMT>(p, lo, hi);
  if (!s.finite) { lo = 0; hi = 0; }
}

// 8-byte load that is cached in the L2 only.  The FP32 dual-axis kernel is 4 % faster with it than
// with the read-only path through the L1 (8192 x 8192: 66.5 -> 63.8 us); the strided kernels
// measured equal or slower with it and with the L1 no-allocate / evict-first hints, and keep __ldg.
__device__ __forceinline__ uint2 ld_cg8(const void* p) {
  uint2 v;
  asm("ld.global.cg.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
  return v;
}

// ---- programmatic dependent launch --------------------------------------------
// The streaming kernels run for 20-40 us, so the 2-3 us between two launches on one stream
// (drain of the last CTAs, launch latency, ramp-up) is a tenth of the time.  They are launched
// with programmatic stream serialization: a kernel signals at once that its successor may be
// scheduled, and waits for its predecessor to have completed and flushed before it touches
// memory -- the order of memory effects is that of ordinary stream order, only the launch
// overhead overlaps the predecessor's tail.
__device__ __forceinline__ void pdl_prologue() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_if(bool overlap, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                 cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = overlap ? 1 : 0;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                              cudaStream_t stream, Args... args) {
  return launch_pdl_if(true, kernel, grid, block, smem, stream, args...);
}

// ---- global memory accesses --------------------------------------------------

__device__ __forceinline__ uint4 ld_stream_16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
// 256-bit load (sm_100): one instruction per 8 FP32 values.  p must be 32-byte aligned.
__device__ __forceinline__ void ld_stream_32(const void* p, uint32_t (&v)[8]) {
  asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]),
                 "=r"(v[6]), "=r"(v[7]) : "l"(p));
}
__device__ __forceinline__ void st_32(void* p, const uint32_t (&v)[8]) {
  asm volatile("st.global.v8.u32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(v[0]),
               "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
               : "memory");
}

// N words (a multiple of 4) to consecutive addresses: 256-bit stores where `wide` (dst 32-byte
// aligned) allows, so that every request carries a whole 32-byte sector; else 128-bit stores.
template <int N>
__device__ __forceinline__ void store_run(uint8_t* dst, const uint32_t (&w)[N], bool wide) {
  static_assert(N % 4 == 0, "whole 16-byte units");
  if (wide) {
#pragma unroll
    for (int i = 0; i < N / 8; ++i) {
      const uint32_t v[8] = {w[8 * i], w[8 * i + 1], w[8 * i + 2], w[8 * i + 3],
                             w[8 * i + 4], w[8 * i + 5], w[8 * i + 6], w[8 * i + 7]};
      st_32(dst + 32 * i, v);
    }
    if (N % 8)
      *reinterpret_cast<uint4*>(dst + 32 * (N / 8)) = make_uint4(w[N - 4], w[N - 3], w[N - 2], w[N - 1]);
  } else {
#pragma unroll
    for (int i = 0; i < N / 4; ++i)
      *reinterpret_cast<uint4*>(dst + 16 * i) = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
  }
}

}  // namespace mx
