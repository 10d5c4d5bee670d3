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

// ---------------------------------------------------------------------------
// Contiguous axis
// ---------------------------------------------------------------------------

// Load 8 consecutive elements as FP32 values.  chunk = index of the 8-element
// group.  ALIGNED32: the FP32 tensor base is 32-byte aligned (256-bit load).
template <int DTYPE, bool ALIGNED32>
__device__ __forceinline__ void load8(const void* in, size_t chunk, float (&v)[8]) {
  if (DTYPE == MX_BF16) {
    const uint4 w = ld_stream_16(reinterpret_cast<const uint4*>(in) + chunk);
    const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(u[i] << 16);  // BF16 widens exactly
      v[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u);
    }
  } else if (ALIGNED32) {
    uint32_t u[8];
    ld_stream_32(reinterpret_cast<const char*>(in) + chunk * 32, u);
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(u[i]);
  } else {
    const uint4* p = reinterpret_cast<const uint4*>(in) + chunk * 2;
    const uint4 a = __ldg(p), b = __ldg(p + 1);
    v[0] = __uint_as_float(a.x); v[1] = __uint_as_float(a.y);
    v[2] = __uint_as_float(a.z); v[3] = __uint_as_float(a.w);
    v[4] = __uint_as_float(b.x); v[5] = __uint_as_float(b.y);
    v[6] = __uint_as_float(b.z); v[7] = __uint_as_float(b.w);
  }
}

// U chunks of 8 elements per thread per iteration, all loads issued before any
// arithmetic so that U * 16 (BF16) or U * 32 (FP32) bytes per thread are in flight.
template <int FMT, int ROUND, int DTYPE, int LAYOUT, bool ALIGNED32, int U>
__global__ void __launch_bounds__(kThreads)
quantize_lastaxis_kernel(const void* __restrict__ in, uint8_t* __restrict__ elems,
                         uint8_t* __restrict__ scales, uint32_t n_chunks, uint32_t kblocks,
                         FastDiv kb_div) {
  constexpr int bits = FmtTraits<FMT>::bits;
  const uint32_t lane4 = threadIdx.x & 3u;  // position of this thread's 8 elements in the block
  const uint32_t span = kThreads * U;
  for (uint32_t base = blockIdx.x * span; base < n_chunks; base += gridDim.x * span) {
    float v[U][8];
    bool ok[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint32_t c = base + u * kThreads + threadIdx.x;
      ok[u] = c < n_chunks;  // whole groups of 4 lanes are in or out: n_chunks % 4 == 0
      if (ok[u]) {
        load8<DTYPE, ALIGNED32>(in, c, v[u]);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) v[u][i] = 0.0f;
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint32_t c = base + u * kThreads + threadIdx.x;
      // Line 1 of Algorithm 1: max |V_i| over the block (8 local values, 4 lanes).
      float amax = absmax_nan(v[u][0], v[u][1]);
#pragma unroll
      for (int i = 2; i < 8; ++i) amax = absmax_nan(amax, v[u][i]);
      amax = absmax_nan(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
      amax = absmax_nan(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 2));
      const BlockScale s = block_scale<FMT>(amax);
      // Lines 3-5: P_i = quantize(V_i / X)
      uint32_t lo, hi;
      cast8<FMT, ROUND>(v[u], s, lo, hi);
      if (bits == 6) {
        // 4 lanes hold 6 bytes each; lanes 0..2 of the group store 8 bytes each.
        const uint64_t mine = (uint64_t)lo | ((uint64_t)hi << 32);
        const uint32_t nlo = __shfl_down_sync(0xFFFFFFFFu, lo, 1);
        const uint32_t nhi = __shfl_down_sync(0xFFFFFFFFu, hi, 1);
        const uint64_t next = (uint64_t)nlo | ((uint64_t)nhi << 32);
        const uint64_t q = (mine >> (16 * lane4)) | (next << (48 - 16 * lane4));
        if (ok[u] && lane4 < 3) {
          uint8_t* dst = elems + (size_t)(c >> 2) * 24 + lane4 * 8;
          *reinterpret_cast<uint2*>(dst) = make_uint2((uint32_t)q, (uint32_t)(q >> 32));
        }
      } else if (ok[u]) {
        if (bits == 8) *reinterpret_cast<uint2*>(elems + (size_t)c * 8) = make_uint2(lo, hi);
        else *reinterpret_cast<uint32_t*>(elems + (size_t)c * 4) = lo;
      }
      if (ok[u] && lane4 == 0) {
        const uint32_t blk = c >> 2;
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

template <int FMT, int ROUND, int DTYPE, int LAYOUT>
static cudaError_t launch_lastaxis(const QuantizeArgs& a) {
  constexpr int U = 4;
  const uint32_t n_chunks = (uint32_t)(a.numel / 8);
  const uint32_t kblocks = (uint32_t)(a.L / kBlock);
  const uint32_t span = kThreads * U;
  uint32_t grid = (n_chunks + span - 1) / span;
  const uint32_t cap = (uint32_t)a.sm_count * 8;
  if (grid > cap) grid = cap;
  const FastDiv kd = make_fastdiv(kblocks);
  const bool al32 = DTYPE == MX_F32 && ((uintptr_t)a.in % 32 == 0);
  if (al32)
    quantize_lastaxis_kernel<FMT, ROUND, DTYPE, LAYOUT, true, U><<<grid, kThreads, 0, a.stream>>>(
        a.in, a.elems, a.scales, n_chunks, kblocks, kd);
  else
    quantize_lastaxis_kernel<FMT, ROUND, DTYPE, LAYOUT, false, U><<<grid, kThreads, 0, a.stream>>>(
        a.in, a.elems, a.scales, n_chunks, kblocks, kd);
  return cudaGetLastError();
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
