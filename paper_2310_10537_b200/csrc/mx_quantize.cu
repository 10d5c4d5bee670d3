// Float -> MX conversion kernels (Algorithm 1, Section 3 of arXiv 2310.10537).
//
//   quantize_lastaxis_kernel  blocks run along the contiguous axis: a pure
//                             stream, 8 elements per thread, 4 lanes per block.
//   quantize_strided_kernel   blocks run along a strided axis (the transposed
//                             operands of dgrad / wgrad, Section 4.1): each
//                             thread owns whole blocks of a few columns, reads
//                             rows coalesced across the warp and writes the
//                             result with the block axis innermost.
//
// Both are bound by HBM bandwidth: in_bytes + bits/8 + 1/32 bytes per element.
#include "mx_device.cuh"
#include "mx_launch.h"

namespace mx {

constexpr int kThreads = 256;
#ifndef MX_Q_U
#define MX_Q_U 1      // 64-byte units per thread and loop iteration
#endif
#ifndef MX_Q_CAP
#define MX_Q_CAP 0     // CTAs per SM the grid is capped at (0 = no cap, -1 = resident CTAs)
#endif
#ifndef MX_Q_MINB
#define MX_Q_MINB 4   // resident CTAs per SM the register allocation must allow
#endif

// ---------------------------------------------------------------------------
// Contiguous axis
// ---------------------------------------------------------------------------

// A thread owns 64 bytes of input: one whole block of BF16 (32 elements) or half
// a block of FP32 (16 elements, the other half in the neighbouring lane).  It
// reads them with two 256-bit loads (four 128-bit loads when the tensor is only
// 16-byte aligned), so a block needs at most one shuffle, the scale is computed
// once per 64 bytes, and the codes leave as one 32 / 16-byte store.
template <int DTYPE> struct LastAxis {
  static constexpr int kElems = DTYPE == MX_BF16 ? 32 : 16;  // elements per thread
  static constexpr int kLanes = kBlock / kElems;             // lanes per MX block
};

template <int DTYPE, bool ALIGNED32>
__device__ __forceinline__ void load_unit(const void* in, size_t unit,
                                          float (&v)[LastAxis<DTYPE>::kElems]) {
  uint32_t w[16];
  const char* p = reinterpret_cast<const char*>(in) + unit * 64;
  if (ALIGNED32) {
    uint32_t a[8], b[8];
    ld_stream_32(p, a);
    ld_stream_32(p + 32, b);
#pragma unroll
    for (int i = 0; i < 8; ++i) { w[i] = a[i]; w[8 + i] = b[i]; }
  } else {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint4 q = ld_stream_16(p + 16 * j);
      w[4 * j] = q.x; w[4 * j + 1] = q.y; w[4 * j + 2] = q.z; w[4 * j + 3] = q.w;
    }
  }
  if (DTYPE == MX_BF16) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      v[(2 * i) % LastAxis<DTYPE>::kElems] = __uint_as_float(w[i] << 16);  // BF16 widens exactly
      v[(2 * i + 1) % LastAxis<DTYPE>::kElems] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  } else {
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i % LastAxis<DTYPE>::kElems] = __uint_as_float(w[i]);
  }
}

template <int FMT, int ROUND, int DTYPE, int LAYOUT, bool ALIGNED32, int U>
__global__ void __launch_bounds__(kThreads, MX_Q_MINB)
quantize_lastaxis_kernel(const void* __restrict__ in, uint8_t* __restrict__ elems,
                         uint8_t* __restrict__ scales, uint32_t n_units, uint32_t kblocks,
                         FastDiv kb_div, uint32_t scale_words) {
  constexpr int bits = FmtTraits<FMT>::bits;
  constexpr int kElems = LastAxis<DTYPE>::kElems;
  constexpr int kLanes = LastAxis<DTYPE>::kLanes;
  constexpr int kOutBytes = kElems * bits / 8;  // 32/24/16 (BF16) or 16/12/8 (FP32) per thread
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t span = kThreads * U;
  for (uint32_t base = blockIdx.x * span; base < n_units; base += gridDim.x * span) {
    float v[U][kElems];
    bool ok[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint32_t unit = base + u * kThreads + threadIdx.x;
      ok[u] = unit < n_units;  // groups of 4 blocks are in or out together: n_units * kLanes % 4 == 0 or tail
      if (ok[u]) {
        load_unit<DTYPE, ALIGNED32>(in, unit, v[u]);
      } else {
#pragma unroll
        for (int i = 0; i < kElems; ++i) v[u][i] = 0.0f;
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint32_t unit = base + u * kThreads + threadIdx.x;
      // Line 1 of Algorithm 1: max |V_i| over the block
      float amax = absmax_nan(v[u][0], v[u][1]);
#pragma unroll
      for (int i = 2; i < kElems; ++i) amax = absmax_nan(amax, v[u][i]);
      if (kLanes == 2) amax = absmax_nan(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
      const BlockScale s = block_scale<FMT>(amax);
      // Lines 3-5: P_i = quantize(V_i / X)
      uint32_t w[kElems / 4];  // 8-bit: all words; 6-bit: 3 of every 4; 4-bit: every other
#pragma unroll
      for (int g = 0; g < kElems / 8; ++g) {
        float x[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) x[i] = v[u][8 * g + i];
        cast8<FMT, ROUND>(x, s, w[2 * g], w[2 * g + 1]);
      }
      uint8_t* dst = elems + (size_t)unit * kOutBytes;
      if (bits == 8) {
        if (kElems == 32) {
          if (ok[u]) {
            if (ALIGNED32) {
              const uint32_t o[8] = {w[0], w[1], w[2], w[3], w[4 % (kElems / 4)], w[5 % (kElems / 4)],
                                     w[6 % (kElems / 4)], w[7 % (kElems / 4)]};
              st_32(dst, o);
            } else {
              reinterpret_cast<uint4*>(dst)[0] = make_uint4(w[0], w[1], w[2], w[3]);
              reinterpret_cast<uint4*>(dst)[1] = make_uint4(w[4 % (kElems / 4)], w[5 % (kElems / 4)],
                                                            w[6 % (kElems / 4)], w[7 % (kElems / 4)]);
            }
          }
        } else if (ok[u]) {
          *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      } else if (bits == 4) {
        if (kElems == 32) {
          if (ok[u]) *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[2], w[4 % (kElems / 4)], w[6 % (kElems / 4)]);
        } else if (ok[u]) {
          *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[2]);
        }
      } else {
        // 6-bit: each group of 8 codes is 48 bits (lo 32 + hi 16)
        const uint64_t g0 = (uint64_t)w[0] | ((uint64_t)w[1] << 32);
        const uint64_t g1 = (uint64_t)w[2] | ((uint64_t)w[3] << 32);
        if (kElems == 32) {
          const uint64_t g2 = (uint64_t)w[4 % (kElems / 4)] | ((uint64_t)w[5 % (kElems / 4)] << 32);
          const uint64_t g3 = (uint64_t)w[6 % (kElems / 4)] | ((uint64_t)w[7 % (kElems / 4)] << 32);
          const uint64_t q0 = g0 | (g1 << 48), q1 = (g1 >> 16) | (g2 << 32), q2 = (g2 >> 32) | (g3 << 16);
          if (ok[u]) {
            uint2* d2 = reinterpret_cast<uint2*>(dst);  // 24-byte blocks are 8-byte aligned
            d2[0] = make_uint2((uint32_t)q0, (uint32_t)(q0 >> 32));
            d2[1] = make_uint2((uint32_t)q1, (uint32_t)(q1 >> 32));
            d2[2] = make_uint2((uint32_t)q2, (uint32_t)(q2 >> 32));
          }
        } else {
          // 12 bytes per lane, 24 per block: the even lane stores bytes 0..15, the odd lane 16..23
          const uint32_t t0 = (uint32_t)g0, t1 = (uint32_t)(g0 >> 32) | ((uint32_t)g1 << 16),
                         t2 = (uint32_t)(g1 >> 16);
          const uint32_t n0 = __shfl_down_sync(0xFFFFFFFFu, t0, 1);
          if (ok[u]) {
            uint8_t* blk = elems + (size_t)(unit >> 1) * 24;
            if ((lane & 1u) == 0) {
              reinterpret_cast<uint2*>(blk)[0] = make_uint2(t0, t1);
              reinterpret_cast<uint2*>(blk)[1] = make_uint2(t2, n0);
            } else {
              reinterpret_cast<uint2*>(blk)[2] = make_uint2(t1, t2);
            }
          }
        }
      }
      // scale bytes: four consecutive blocks of a row share one 32-bit word
      const uint32_t blk = unit / kLanes;
      if (scale_words) {
        uint32_t word = s.byte << (8 * (blk & 3u));
        word |= __shfl_xor_sync(0xFFFFFFFFu, word, kLanes);
        word |= __shfl_xor_sync(0xFFFFFFFFu, word, 2 * kLanes);
        if (ok[u] && (lane & (4 * kLanes - 1)) == 0) {
          size_t off;
          if (LAYOUT == MX_SCALES_LINEAR) {
            off = blk;
          } else {
            const uint32_t row = fastdiv(blk, kb_div);
            off = scale_offset<LAYOUT>(row, blk - row * kblocks, kblocks);
          }
          *reinterpret_cast<uint32_t*>(scales + off) = word;
        }
      } else if (ok[u] && (lane & (kLanes - 1)) == 0) {
        size_t off;
        if (LAYOUT == MX_SCALES_LINEAR) {
          off = blk;
        } else {
          const uint32_t row = fastdiv(blk, kb_div);
          off = scale_offset<LAYOUT>(row, blk - row * kblocks, kblocks);
        }
        scales[off] = (uint8_t)s.byte;
      }
    }
  }
}

// ---------------------------------------------------------------------------
// Strided axis
// ---------------------------------------------------------------------------

// Tensor viewed as [outer, L, inner], blocks along L.  A thread owns COLS
// adjacent columns (inner positions) and walks KB_PER_THREAD consecutive blocks;
// a warp therefore reads 32*COLS consecutive elements of each input row.
// Output row = o * inner + column, block axis innermost.
template <int FMT, int ROUND, int DTYPE, int LAYOUT, int COLS>
__global__ void __launch_bounds__(kThreads)
quantize_strided_kernel(const void* __restrict__ in, uint8_t* __restrict__ elems,
                        uint8_t* __restrict__ scales, uint32_t outer, uint32_t L,
                        uint32_t inner, uint32_t kb_per_thread) {
  constexpr int bits = FmtTraits<FMT>::bits;
  const uint32_t kblocks = L / kBlock;
  const uint32_t col0 = (blockIdx.x * kThreads + threadIdx.x) * COLS;
  if (col0 >= inner) return;  // no warp-level exchange in this kernel
  const uint32_t kb_begin = blockIdx.y * kb_per_thread;
  const uint32_t kb_end = min(kb_begin + kb_per_thread, kblocks);
  const size_t esz = DTYPE == MX_BF16 ? 2 : 4;
  const size_t row_pitch = (size_t)inner * esz;
  const size_t out_row_bytes = (size_t)L * bits / 8;

  for (uint32_t o = blockIdx.z; o < outer; o += gridDim.z)
  for (uint32_t kb = kb_begin; kb < kb_end; ++kb) {
    const char* src = reinterpret_cast<const char*>(in) + ((size_t)o * L * inner + col0) * esz;
    // 32 input rows x COLS columns, every load issued before the arithmetic
    float v[COLS][kBlock];
    const char* p = src + (size_t)kb * kBlock * row_pitch;
#pragma unroll
    for (int k = 0; k < kBlock; ++k) {
      const char* q = p + (size_t)k * row_pitch;
      if (DTYPE == MX_BF16) {
        if (COLS == 4) {
          const uint2 w = __ldg(reinterpret_cast<const uint2*>(q));
          v[0][k] = __uint_as_float(w.x << 16); v[1 % COLS][k] = __uint_as_float(w.x & 0xFFFF0000u);
          v[2 % COLS][k] = __uint_as_float(w.y << 16); v[3 % COLS][k] = __uint_as_float(w.y & 0xFFFF0000u);
        } else if (COLS == 2) {
          const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(q));
          v[0][k] = __uint_as_float(w << 16); v[1 % COLS][k] = __uint_as_float(w & 0xFFFF0000u);
        } else {
          v[0][k] = __uint_as_float((uint32_t)__ldg(reinterpret_cast<const uint16_t*>(q)) << 16);
        }
      } else {
        if (COLS == 4) {
          const float4 w = __ldg(reinterpret_cast<const float4*>(q));
          v[0][k] = w.x; v[1 % COLS][k] = w.y; v[2 % COLS][k] = w.z; v[3 % COLS][k] = w.w;
        } else if (COLS == 2) {
          const float2 w = __ldg(reinterpret_cast<const float2*>(q));
          v[0][k] = w.x; v[1 % COLS][k] = w.y;
        } else {
          v[0][k] = __ldg(reinterpret_cast<const float*>(q));
        }
      }
    }
#pragma unroll
    for (int c = 0; c < COLS; ++c) {
      float amax = absmax_nan(v[c][0], v[c][1]);
#pragma unroll
      for (int k = 2; k < kBlock; ++k) amax = absmax_nan(amax, v[c][k]);
      const BlockScale s = block_scale<FMT>(amax);
      const uint32_t row = o * inner + col0 + c;
      uint8_t* dst = elems + (size_t)row * out_row_bytes + (size_t)kb * (kBlock * bits / 8);
      uint32_t w[8];
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        float x[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) x[i] = v[c][g * 8 + i];
        cast8<FMT, ROUND>(x, s, w[2 * g], w[2 * g + 1]);
      }
      if (bits == 8) {
        reinterpret_cast<uint4*>(dst)[0] = make_uint4(w[0], w[1], w[2], w[3]);
        reinterpret_cast<uint4*>(dst)[1] = make_uint4(w[4], w[5], w[6], w[7]);
      } else if (bits == 4) {
        reinterpret_cast<uint4*>(dst)[0] = make_uint4(w[0], w[2], w[4], w[6]);
      } else {
        // four 48-bit groups -> 24 bytes
        const uint64_t g0 = (uint64_t)w[0] | ((uint64_t)w[1] << 32);
        const uint64_t g1 = (uint64_t)w[2] | ((uint64_t)w[3] << 32);
        const uint64_t g2 = (uint64_t)w[4] | ((uint64_t)w[5] << 32);
        const uint64_t g3 = (uint64_t)w[6] | ((uint64_t)w[7] << 32);
        const uint64_t q0 = g0 | (g1 << 48), q1 = (g1 >> 16) | (g2 << 32), q2 = (g2 >> 32) | (g3 << 16);
        uint2* d2 = reinterpret_cast<uint2*>(dst);
        d2[0] = make_uint2((uint32_t)q0, (uint32_t)(q0 >> 32));
        d2[1] = make_uint2((uint32_t)q1, (uint32_t)(q1 >> 32));
        d2[2] = make_uint2((uint32_t)q2, (uint32_t)(q2 >> 32));
      }
      scales[scale_offset<LAYOUT>(row, kb, kblocks)] = (uint8_t)s.byte;
    }
  }
}

// ---------------------------------------------------------------------------
// Host-side dispatch
// ---------------------------------------------------------------------------

// Resident CTAs per SM of a kernel (queried once per instantiation): persistent grids are sized
// to exactly fill the machine so that no partial wave trails the launch.
template <typename K>
static int resident_ctas(K kernel, int threads) {
  int n = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, threads, 0) != cudaSuccess || n < 1) n = 1;
  return n;
}

template <int FMT, int ROUND, int DTYPE, int LAYOUT, bool AL32>
static cudaError_t launch_lastaxis_al(const QuantizeArgs& a) {
  constexpr int U = MX_Q_U;
  constexpr int kElems = LastAxis<DTYPE>::kElems;
  const uint32_t n_units = (uint32_t)(a.numel / kElems);
  const uint32_t n_blocks = (uint32_t)(a.numel / kBlock);
  const uint32_t kblocks = (uint32_t)(a.L / kBlock);
  const uint32_t span = kThreads * U;
  auto kernel = quantize_lastaxis_kernel<FMT, ROUND, DTYPE, LAYOUT, AL32, U>;
  uint32_t grid = (n_units + span - 1) / span;
#if MX_Q_CAP > 0
  const uint32_t cap = (uint32_t)a.sm_count * MX_Q_CAP;
  if (grid > cap) grid = cap;
#elif MX_Q_CAP < 0
  static const int per_sm = resident_ctas(kernel, kThreads);
  const uint32_t cap = (uint32_t)(a.sm_count * per_sm);
  if (grid > cap) grid = cap;
#endif
  const FastDiv kd = make_fastdiv(kblocks);
  // one 32-bit store per four scale bytes when groups of four never straddle a row or the end
  const uint32_t scale_words = LAYOUT == MX_SCALES_LINEAR ? (n_blocks % 4 == 0) : (kblocks % 4 == 0);
  kernel<<<grid, kThreads, 0, a.stream>>>(a.in, a.elems, a.scales, n_units, kblocks, kd, scale_words);
  return cudaGetLastError();
}

template <int FMT, int ROUND, int DTYPE, int LAYOUT>
static cudaError_t launch_lastaxis(const QuantizeArgs& a) {
  if ((uintptr_t)a.in % 32 == 0 && (uintptr_t)a.elems % 32 == 0)
    return launch_lastaxis_al<FMT, ROUND, DTYPE, LAYOUT, true>(a);
  return launch_lastaxis_al<FMT, ROUND, DTYPE, LAYOUT, false>(a);
}

template <int FMT, int ROUND, int DTYPE, int LAYOUT, int COLS>
static cudaError_t launch_strided_cols(const QuantizeArgs& a) {
  const uint32_t kblocks = (uint32_t)(a.L / kBlock);
  const uint32_t threads_x = (uint32_t)((a.inner + COLS - 1) / COLS);
  const uint32_t kb_per_thread = kblocks < 4 ? kblocks : 4;
  dim3 grid((threads_x + kThreads - 1) / kThreads, (kblocks + kb_per_thread - 1) / kb_per_thread,
            (uint32_t)(a.outer < 65535 ? a.outer : 65535));
  quantize_strided_kernel<FMT, ROUND, DTYPE, LAYOUT, COLS><<<grid, kThreads, 0, a.stream>>>(
      a.in, a.elems, a.scales, (uint32_t)a.outer, (uint32_t)a.L, (uint32_t)a.inner, kb_per_thread);
  return cudaGetLastError();
}

template <int FMT, int ROUND, int DTYPE, int LAYOUT>
static cudaError_t launch_strided(const QuantizeArgs& a) {
  // widest column group whose loads stay aligned: 8 bytes per row and thread
  const int wide = DTYPE == MX_BF16 ? 4 : 2;
  if (a.inner % wide == 0 && (uintptr_t)a.in % 8 == 0)
    return launch_strided_cols<FMT, ROUND, DTYPE, LAYOUT, (DTYPE == MX_BF16 ? 4 : 2)>(a);
  return launch_strided_cols<FMT, ROUND, DTYPE, LAYOUT, 1>(a);
}

template <int FMT, int ROUND, int DTYPE, int LAYOUT>
static cudaError_t launch_any(const QuantizeArgs& a) {
  if (a.inner == 1) return launch_lastaxis<FMT, ROUND, DTYPE, LAYOUT>(a);
  return launch_strided<FMT, ROUND, DTYPE, LAYOUT>(a);
}

template <int FMT, int ROUND>
static cudaError_t dispatch_dtype_layout(const QuantizeArgs& a) {
  if (a.dtype == MX_BF16) {
    return a.layout == MX_SCALES_LINEAR ? launch_any<FMT, ROUND, MX_BF16, MX_SCALES_LINEAR>(a)
                                        : launch_any<FMT, ROUND, MX_BF16, MX_SCALES_SWIZZLED>(a);
  }
  return a.layout == MX_SCALES_LINEAR ? launch_any<FMT, ROUND, MX_F32, MX_SCALES_LINEAR>(a)
                                      : launch_any<FMT, ROUND, MX_F32, MX_SCALES_SWIZZLED>(a);
}

template <int FMT>
static cudaError_t dispatch_round(const QuantizeArgs& a) {
  return a.rounding == MX_RHAZ ? dispatch_dtype_layout<FMT, MX_RHAZ>(a)
                               : dispatch_dtype_layout<FMT, MX_RNE>(a);
}

cudaError_t launch_quantize(const QuantizeArgs& a) {
  switch (a.fmt) {
    case MX_E4M3: return dispatch_round<MX_E4M3>(a);
    case MX_E5M2: return dispatch_round<MX_E5M2>(a);
    case MX_E3M2: return dispatch_round<MX_E3M2>(a);
    case MX_E2M3: return dispatch_round<MX_E2M3>(a);
    case MX_E2M1: return dispatch_round<MX_E2M1>(a);
    default: return dispatch_round<MX_INT8>(a);
  }
}

}  // namespace mx
