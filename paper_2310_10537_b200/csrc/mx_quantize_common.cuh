// Pieces shared by the quantize kernels (contiguous axis, strided axis, dual axis): block maxima
// over packed registers and element access into packed rows.
#pragma once

#include "mx_device.cuh"

namespace mx {

// max |V_i| over the unit as a balanced tree (short dependency chains), on packed BF16 pairs
// where the input is BF16.
template <int DTYPE>
__device__ __forceinline__ float unit_amax(const uint32_t (&w)[16]) {
  if constexpr (DTYPE == MX_BF16) {
    uint32_t m[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) m[i] = absmax_nan_bf16x2(w[2 * i], w[2 * i + 1]);
#pragma unroll
    for (int i = 0; i < 4; ++i) m[i] = absmax_nan_bf16x2(m[2 * i], m[2 * i + 1]);
    m[0] = absmax_nan_bf16x2(absmax_nan_bf16x2(m[0], m[1]), absmax_nan_bf16x2(m[2], m[3]));
    return bf16x2_halves_max(m[0]);
  } else {
    float m[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) m[i] = absmax_nan(__uint_as_float(w[2 * i]), __uint_as_float(w[2 * i + 1]));
#pragma unroll
    for (int i = 0; i < 4; ++i) m[i] = absmax_nan(m[2 * i], m[2 * i + 1]);
    return absmax_nan(absmax_nan(m[0], m[1]), absmax_nan(m[2], m[3]));
  }
}

// Elements 8g .. 8g+7 of the unit as FP32 values.
template <int DTYPE>
__device__ __forceinline__ void unit_group(const uint32_t (&w)[16], int g, float (&x)[8]) {
  if (DTYPE == MX_BF16) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[2 * i] = __uint_as_float(imad(w[4 * g + i], 1u << 16, 0u));  // BF16 widens exactly (shift on the multiply-add unit)
      x[2 * i + 1] = __uint_as_float(w[4 * g + i] & 0xFFFF0000u);
    }
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] = __uint_as_float(w[(8 * g + i) % 16]);
  }
}

template <int DTYPE, int COLS> struct StridedRow {
  static constexpr int kBytes = COLS * (DTYPE == MX_BF16 ? 2 : 4);   // bytes loaded per row: 8, 4 or 2
  static constexpr int kWords = kBytes >= 4 ? kBytes / 4 : 1;
};

// Element (row k, column c) of the packed rows as an FP32 value.
template <int DTYPE, int COLS>
__device__ __forceinline__ float strided_elem(const uint32_t (&raw)[kBlock][StridedRow<DTYPE, COLS>::kWords],
                                              int k, int c) {
  if (DTYPE == MX_BF16) {
    const uint32_t w = raw[k][(c / 2) % StridedRow<DTYPE, COLS>::kWords];
    return __uint_as_float((c & 1) ? (w & 0xFFFF0000u) : imad(w, 1u << 16, 0u));
  }
  return __uint_as_float(raw[k][c % StridedRow<DTYPE, COLS>::kWords]);
}


// amax of every column of a thread's 32 packed rows (Line 1 of Algorithm 1 for COLS blocks at
// once): balanced trees, on packed BF16 pairs (two columns per operation) where the input is BF16.
template <int DTYPE, int COLS>
__device__ __forceinline__ void column_amax(const uint32_t (&raw)[kBlock][StridedRow<DTYPE, COLS>::kWords],
                                            float (&amax)[COLS]) {
  constexpr int kWords = StridedRow<DTYPE, COLS>::kWords;
  if (DTYPE == MX_BF16) {
#pragma unroll
    for (int wi = 0; wi < kWords; ++wi) {
      uint32_t m[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) m[i] = absmax_nan_bf16x2(raw[2 * i][wi], raw[2 * i + 1][wi]);
#pragma unroll
      for (int n = 8; n >= 1; n >>= 1)
#pragma unroll
        for (int i = 0; i < n; ++i) m[i] = absmax_nan_bf16x2(m[2 * i], m[2 * i + 1]);
      amax[(2 * wi) % COLS] = __uint_as_float((m[0] << 16) & 0x7FFF0000u);
      if (COLS > 1) amax[(2 * wi + 1) % COLS] = __uint_as_float(m[0] & 0x7FFF0000u);
    }
  } else {
#pragma unroll
    for (int c = 0; c < COLS; ++c) {
      float m[16];
#pragma unroll
      for (int i = 0; i < 16; ++i)
        m[i] = absmax_nan(__uint_as_float(raw[2 * i][c % kWords]), __uint_as_float(raw[2 * i + 1][c % kWords]));
#pragma unroll
      for (int n = 8; n >= 1; n >>= 1)
#pragma unroll
        for (int i = 0; i < n; ++i) m[i] = absmax_nan(m[2 * i], m[2 * i + 1]);
      amax[c] = m[0];
    }
  }
}

// Codes of one column block (32 rows of column c) as eight words in cast8's layout.
template <int FMT, int ROUND, int DTYPE, int COLS>
__device__ __forceinline__ void column_cast(const uint32_t (&raw)[kBlock][StridedRow<DTYPE, COLS>::kWords],
                                            int c, const BlockScale& s, uint32_t (&w)[8]) {
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    float x[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] = strided_elem<DTYPE, COLS>(raw, g * 8 + i, c);
    cast8<FMT, ROUND>(x, s, w[2 * g], w[2 * g + 1]);
  }
}

// The 24 bytes of a 6-bit block from cast8's four (32 + 16)-bit groups, as six words: joins of
// disjoint fields go through the multiply-add unit or one byte permute (see pack8).
__device__ __forceinline__ void pack6_words(const uint32_t (&w)[8], uint32_t (&o)[6]) {
  o[0] = w[0];
  o[1] = imad(w[2], 1u << 16, w[1]);          // w[1] holds 16 bits
  o[2] = __byte_perm(w[2], w[3], 0x5432);     // (w[2] >> 16) | (w[3] << 16)
  o[3] = w[4];
  o[4] = imad(w[6], 1u << 16, w[5]);
  o[5] = __byte_perm(w[6], w[7], 0x5432);
}
__device__ __forceinline__ void pack6(const uint32_t (&w)[8], uint64_t& q0, uint64_t& q1, uint64_t& q2) {
  uint32_t o[6];
  pack6_words(w, o);
  q0 = (uint64_t)o[0] | ((uint64_t)o[1] << 32);
  q1 = (uint64_t)o[2] | ((uint64_t)o[3] << 32);
  q2 = (uint64_t)o[4] | ((uint64_t)o[5] << 32);
}

}  // namespace mx
