// Float -> MX conversion kernels (Algorithm 1, Section 3 of arXiv 2310.10537).
//
//   quantize_lastaxis_kernel        blocks run along the contiguous axis: a pure stream, 64 bytes
//                                   of input per thread (a whole BF16 block, half an FP32 block).
//   quantize_strided_kernel         blocks run along a strided axis (the transposed operands of
//                                   dgrad / wgrad, Section 4.1): a thread owns whole blocks of a
//                                   few adjacent columns, rows are read coalesced across the warp
//                                   and the result is written with the block axis innermost.
//   quantize_strided_staged_kernel  the same for 6- and 4-bit codes, whose output runs are gathered
//                                   in shared memory so that they leave as whole 32-byte sectors.
//
// All are bound by HBM bandwidth: in_bytes + bits/8 + 1/32 bytes per element.
#include "mx_device.cuh"
#include "mx_launch.h"
#include "mx_quantize_common.cuh"

namespace mx {

constexpr int kThreads = 256;
constexpr int kUnitsPerThread = 1;  // 64-byte units per thread (more only lowered occupancy)
constexpr int kMinCtasPerSm = 4;    // resident CTAs per SM the register allocation must allow

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

// Raw 64 bytes of a unit as sixteen 32-bit words.
template <bool ALIGNED32>
__device__ __forceinline__ void load_unit(const void* in, size_t unit, uint32_t (&w)[16]) {
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
}

template <int FMT, int ROUND, int DTYPE, int LAYOUT, bool ALIGNED32, int U>
__global__ void __launch_bounds__(kThreads, kMinCtasPerSm)
quantize_lastaxis_kernel(const void* __restrict__ in, uint8_t* __restrict__ elems,
                         uint8_t* __restrict__ scales, uint32_t n_units, uint32_t kblocks,
                         FastDiv kb_div, uint32_t scale_words) {
  constexpr int bits = FmtTraits<FMT>::bits;
  constexpr int kElems = LastAxis<DTYPE>::kElems;
  constexpr int kLanes = LastAxis<DTYPE>::kLanes;
  constexpr int kOutBytes = kElems * bits / 8;  // 32/24/16 (BF16) or 16/12/8 (FP32) per thread
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t span = kThreads * U;
  pdl_prologue();
  for (uint32_t base = blockIdx.x * span; base < n_units; base += gridDim.x * span) {
    uint32_t raw[U][16];
    bool ok[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint32_t unit = base + u * kThreads + threadIdx.x;
      ok[u] = unit < n_units;  // groups of 4 blocks are in or out together: n_units * kLanes % 4 == 0 or tail
      if (ok[u]) {
        load_unit<ALIGNED32>(in, unit, raw[u]);
      } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) raw[u][i] = 0u;
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint32_t unit = base + u * kThreads + threadIdx.x;
      // Line 1 of Algorithm 1: max |V_i| over the block
      float amax = unit_amax<DTYPE>(raw[u]);
      if (kLanes == 2) amax = absmax_nan(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
      const BlockScale s = block_scale<FMT>(amax);
      // Lines 3-5: P_i = quantize(V_i / X)
      uint32_t w[kElems / 4];  // 8-bit: all words; 6-bit: 3 of every 4; 4-bit: every other
      // INT8: the saturation at +-127 can only bite where the block maximum scales to 127.5 or more
      // (one block in ~180 for smooth data); a warp none of whose blocks does skips the per-element
      // clamp, which sits on the kernel's busiest pipe
      bool saturating = true;
      if (FMT == MX_INT8) {
        // what the cast makes of the largest element, without its sign (amax carries an arbitrary one)
        float top = fabsf(mul_ftz(amax, s.m1) * s.m2);
        if (ROUND == MX_RHAZ) top = __uint_as_float(__float_as_uint(top) | 1u);  // (the sticky bit of ties-away)
        saturating = __any_sync(0xFFFFFFFFu, !(top < 127.5f));
      }
      if (FMT != MX_INT8 || saturating) {
#pragma unroll
        for (int g = 0; g < kElems / 8; ++g) {
          float x[8];
          unit_group<DTYPE>(raw[u], g, x);
          cast8<FMT, ROUND>(x, s, w[2 * g], w[2 * g + 1]);
        }
      } else {
#pragma unroll
        for (int g = 0; g < kElems / 8; ++g) {
          float x[8];
          unit_group<DTYPE>(raw[u], g, x);
          cast8<FMT, ROUND, false>(x, s, w[2 * g], w[2 * g + 1]);
        }
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
        if (kElems == 32) {
          const uint32_t cw[8] = {w[0], w[1], w[2], w[3], w[4 % (kElems / 4)], w[5 % (kElems / 4)],
                                  w[6 % (kElems / 4)], w[7 % (kElems / 4)]};
          uint32_t o[6];
          pack6_words(cw, o);
          if (ok[u]) {
            uint2* d2 = reinterpret_cast<uint2*>(dst);  // 24-byte blocks are 8-byte aligned
            d2[0] = make_uint2(o[0], o[1]);
            d2[1] = make_uint2(o[2], o[3]);
            d2[2] = make_uint2(o[4], o[5]);
          }
        } else {
          // 12 bytes per lane, 24 per block: the even lane stores bytes 0..15, the odd lane 16..23
          const uint32_t t0 = w[0], t1 = imad(w[2], 1u << 16, w[1]), t2 = __byte_perm(w[2], w[3], 0x5432);
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

// Tensor viewed as [outer, L, inner], blocks along L.  A thread owns COLS adjacent
// columns (inner positions) and walks kb_per_thread consecutive blocks; a warp therefore
// reads 32*COLS consecutive elements of each input row.  The 32 rows of a block stay in
// registers in their packed input form (8 bytes per row for the wide variants: four BF16
// or two FP32 columns), so a block of every column is complete in one thread: no shared
// memory, no shuffles.  Output row = o * inner + column, block axis innermost.
constexpr int kStridedThreads = 128;

// 8 bytes of a row.  ONE_WAVE: the whole grid is resident at once, so every warp issues its 32 row
// loads at the same moment and the lines they would allocate exceed the L1 (FP32 4096 x 4096 -> 6-bit:
// 15.2 -> 14.4 us without allocation); in a grid of several waves the warps are staggered and the
// allocating read-only path is the faster one (8192 x 8192: 50.4 against 52.8 us).
template <bool ONE_WAVE>
__device__ __forceinline__ uint2 ld_row8(const char* q) {
  if (ONE_WAVE) {
    uint2 v;
    asm("ld.global.nc.L1::no_allocate.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(q));
    return v;
  }
  return __ldg(reinterpret_cast<const uint2*>(q));
}

template <int FMT, int ROUND, int DTYPE, int LAYOUT, int COLS, bool ONE_WAVE = false>
__global__ void __launch_bounds__(kStridedThreads, 4)
quantize_strided_kernel(const void* __restrict__ in, uint8_t* __restrict__ elems,
                        uint8_t* __restrict__ scales, uint32_t outer, uint32_t L,
                        uint32_t inner, uint32_t kb_per_thread) {
  constexpr int bits = FmtTraits<FMT>::bits;
  constexpr int kWords = StridedRow<DTYPE, COLS>::kWords;
  constexpr int kRowBytes = StridedRow<DTYPE, COLS>::kBytes;
  const uint32_t kblocks = L / kBlock;
  const uint32_t col0 = (blockIdx.x * kStridedThreads + threadIdx.x) * COLS;
  pdl_prologue();
  if (col0 >= inner) return;  // no warp-level exchange in this kernel
  const uint32_t kb_begin = blockIdx.y * kb_per_thread;
  const uint32_t kb_end = min(kb_begin + kb_per_thread, kblocks);
  const size_t esz = DTYPE == MX_BF16 ? 2 : 4;
  const size_t row_pitch = (size_t)inner * esz;
  const size_t out_row_bytes = (size_t)L * bits / 8;
  const bool al32 = (reinterpret_cast<uintptr_t>(elems) & 31u) == 0;  // 8-bit rows are whole 32-byte units

  for (uint32_t o = blockIdx.z; o < outer; o += gridDim.z)
  for (uint32_t kb = kb_begin; kb < kb_end; ++kb) {
    const char* p = reinterpret_cast<const char*>(in) + ((size_t)o * L * inner + col0) * esz +
                    (size_t)kb * kBlock * row_pitch;
    // 32 input rows, every load issued before the arithmetic
    uint32_t raw[kBlock][kWords];
#pragma unroll
    for (int k = 0; k < kBlock; ++k) {
      const char* q = p + (size_t)k * row_pitch;
      if (kRowBytes == 8) {
        const uint2 w = ld_row8<ONE_WAVE>(q);
        raw[k][0] = w.x; raw[k][1 % kWords] = w.y;
      } else if (kRowBytes == 4) {
        raw[k][0] = __ldg(reinterpret_cast<const uint32_t*>(q));
      } else {
        raw[k][0] = (uint32_t)__ldg(reinterpret_cast<const uint16_t*>(q));
      }
    }
    // Line 1 of Algorithm 1 for every column: balanced trees over the 32 rows, on packed
    // BF16 pairs where the input is BF16 (two columns per operation)
    float amax[COLS];
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
#pragma unroll
    for (int c = 0; c < COLS; ++c) {
      const BlockScale s = block_scale<FMT>(amax[c]);
      const uint32_t row = o * inner + col0 + c;
      uint8_t* dst = elems + (size_t)row * out_row_bytes + (size_t)kb * (kBlock * bits / 8);
      uint32_t w[8];
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        float x[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) x[i] = strided_elem<DTYPE, COLS>(raw, g * 8 + i, c);
        cast8<FMT, ROUND>(x, s, w[2 * g], w[2 * g + 1]);
      }
      if (bits == 8) {
        if (al32) {  // one 256-bit store: a whole sector in a single request
          st_32(dst, w);
        } else {
          reinterpret_cast<uint4*>(dst)[0] = make_uint4(w[0], w[1], w[2], w[3]);
          reinterpret_cast<uint4*>(dst)[1] = make_uint4(w[4], w[5], w[6], w[7]);
        }
      } else if (bits == 4) {
        reinterpret_cast<uint4*>(dst)[0] = make_uint4(w[0], w[2], w[4], w[6]);
      } else {
        uint64_t q0, q1, q2;
        pack6(w, q0, q1, q2);
        uint2* d2 = reinterpret_cast<uint2*>(dst);
        d2[0] = make_uint2((uint32_t)q0, (uint32_t)(q0 >> 32));
        d2[1] = make_uint2((uint32_t)q1, (uint32_t)(q1 >> 32));
        d2[2] = make_uint2((uint32_t)q2, (uint32_t)(q2 >> 32));
      }
      scales[scale_offset<LAYOUT>(row, kb, kblocks)] = (uint8_t)s.byte;
    }
  }
}

// Staged variant of the same kernel for the common case (kblocks % 4 == 0, output rows 16-byte
// aligned): a thread still owns COLS columns, but it walks four consecutive blocks, parks their
// codes in shared memory, and the warp then writes every output row's 128 / 96 / 64-byte run with
// coalesced 32-byte (else 16-byte) stores.  Without this each lane writes its own row and the L2
// sees three (6-bit) or one (4-bit) partial-sector request per block and row, which is what
// bounded the direct version.  Each warp has a private staging area, so only __syncwarp is needed.
constexpr int kStagedThreads = 64;  // resident CTAs per SM below: the measured optimum per variant

template <int FMT, int ROUND, int DTYPE, int LAYOUT, int COLS, bool ONE_WAVE = false>
__global__ void __launch_bounds__(kStagedThreads, (DTYPE == MX_BF16 && FmtTraits<FMT>::bits == 6) ? 6 : 8)
quantize_strided_staged_kernel(const void* __restrict__ in, uint8_t* __restrict__ elems,
                               uint8_t* __restrict__ scales, uint32_t outer, uint32_t L,
                               uint32_t inner) {
  constexpr int bits = FmtTraits<FMT>::bits;
  constexpr int kWords = StridedRow<DTYPE, COLS>::kWords;
  constexpr uint32_t kBpb = kBlock * bits / 8;                     // bytes of one block's codes
  // blocks a CTA walks: four, but two for 4-bit codes -- their two-block run is already a whole
  // sector, and a CTA that lives half as long halves the ragged end of the grid (a fifth of the
  // launch at these sizes)
  constexpr uint32_t NB = bits == 4 ? 2 : 4;
  constexpr uint32_t kSeg = NB * kBpb;                             // the run of a row: 128 / 96 / 64 (32) bytes
  constexpr uint32_t kPitch = kSeg + (bits == 6 ? 8 : 16);         // conflict-free lane stride
  constexpr uint32_t kRows = 32 * COLS;                            // output rows per warp
  extern __shared__ __align__(16) uint8_t staging[];
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint8_t* area = staging + warp * (kRows * kPitch);
  const uint32_t kblocks = L / kBlock;
  const uint32_t warp_col0 = (blockIdx.x * kStagedThreads + warp * 32) * COLS;  // first column of the warp
  pdl_prologue();
  if (warp_col0 >= inner) return;                                  // whole warp out of range
  const uint32_t col0 = warp_col0 + lane * COLS;
  const bool lane_ok = col0 < inner;                               // inner % COLS == 0: all or none of its columns
  const size_t esz = DTYPE == MX_BF16 ? 2 : 4;
  const size_t row_pitch = (size_t)inner * esz;
  const size_t out_row_bytes = (size_t)L * bits / 8;
  const uint32_t rows_here = min(kRows, (inner - warp_col0));      // valid output rows of this warp
  const bool al32 = (reinterpret_cast<uintptr_t>(elems) & 31u) == 0 && out_row_bytes % 32 == 0;

  for (uint32_t o = blockIdx.z; o < outer; o += gridDim.z) {
    const uint32_t kb0 = blockIdx.y * NB;
    uint32_t scale_word[COLS];
#pragma unroll
    for (int c = 0; c < COLS; ++c) scale_word[c] = 0;
#pragma unroll 1
    for (uint32_t j = 0; j < NB; ++j) {
      const uint32_t kb = kb0 + j;
      uint32_t raw[kBlock][kWords];
      if (lane_ok) {
        const char* p = reinterpret_cast<const char*>(in) + ((size_t)o * L * inner + col0) * esz +
                        (size_t)kb * kBlock * row_pitch;
#pragma unroll
        for (int k = 0; k < kBlock; ++k) {
          const uint2 w = ld_row8<ONE_WAVE>(p + (size_t)k * row_pitch);
          raw[k][0] = w.x; raw[k][1 % kWords] = w.y;
        }
      } else {
#pragma unroll
        for (int k = 0; k < kBlock; ++k) { raw[k][0] = 0; raw[k][1 % kWords] = 0; }
      }
      float amax[COLS];
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
          amax[(2 * wi + 1) % COLS] = __uint_as_float(m[0] & 0x7FFF0000u);
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
#pragma unroll
      for (int c = 0; c < COLS; ++c) {
        const BlockScale s = block_scale<FMT>(amax[c]);
        scale_word[c] |= s.byte << (8 * j);
        uint32_t w[8];
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          float x[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) x[i] = strided_elem<DTYPE, COLS>(raw, g * 8 + i, c);
          cast8<FMT, ROUND>(x, s, w[2 * g], w[2 * g + 1]);
        }
        // staging row of (lane, c) is c * 32 + lane: consecutive lanes are one pitch apart
        uint8_t* dst = area + (c * 32 + lane) * kPitch + j * kBpb;
        if (bits == 8) {
          reinterpret_cast<uint4*>(dst)[0] = make_uint4(w[0], w[1], w[2], w[3]);
          reinterpret_cast<uint4*>(dst)[1] = make_uint4(w[4], w[5], w[6], w[7]);
        } else if (bits == 4) {
          reinterpret_cast<uint4*>(dst)[0] = make_uint4(w[0], w[2], w[4], w[6]);
        } else {
          uint64_t q0, q1, q2;
          pack6(w, q0, q1, q2);
          uint2* d2 = reinterpret_cast<uint2*>(dst);  // 8-byte aligned: pitch and 24 j are multiples of 8
          d2[0] = make_uint2((uint32_t)q0, (uint32_t)(q0 >> 32));
          d2[1] = make_uint2((uint32_t)q1, (uint32_t)(q1 >> 32));
          d2[2] = make_uint2((uint32_t)q2, (uint32_t)(q2 >> 32));
        }
      }
    }
    if (lane_ok) {
#pragma unroll
      for (int c = 0; c < COLS; ++c) {  // four scale bytes of a row are one aligned word in both layouts
        const uint32_t row = o * inner + col0 + c;
        uint8_t* sp = scales + scale_offset<LAYOUT>(row, kb0, kblocks);
        if (NB == 4) *reinterpret_cast<uint32_t*>(sp) = scale_word[c];
        else *reinterpret_cast<uint16_t*>(sp) = (uint16_t)scale_word[c];  // kb0 even: two adjacent, aligned bytes
      }
    }
    __syncwarp();
    // write-out, consecutive lanes on consecutive chunks of one output row: 32-byte chunks (one
    // whole sector per request: the L2 request rate bounds this kernel) when the tensor allows
    if (al32) {
      constexpr uint32_t kChunks32 = kSeg / 32;
      for (uint32_t i = lane; i < kRows * kChunks32; i += 32) {
        const uint32_t r = i / kChunks32, ch = i - r * kChunks32;
        const uint32_t c = r >> 5, owner = r & 31;
        const uint32_t col = owner * COLS + c;
        if (col < rows_here) {
          const uint2* src = reinterpret_cast<const uint2*>(area + r * kPitch + ch * 32);
          const uint2 q0 = src[0], q1 = src[1], q2 = src[2], q3 = src[3];
          const uint32_t v[8] = {q0.x, q0.y, q1.x, q1.y, q2.x, q2.y, q3.x, q3.y};
          st_32(elems + (size_t)(o * inner + warp_col0 + col) * out_row_bytes + (size_t)kb0 * kBpb + ch * 32, v);
        }
      }
      __syncwarp();
      continue;
    }
    constexpr uint32_t kChunks = kSeg / 16;
    for (uint32_t i = lane; i < kRows * kChunks; i += 32) {
      const uint32_t r = i / kChunks, ch = i - r * kChunks;      // staging row, chunk in the row
      const uint32_t c = r >> 5, owner = r & 31;                  // column of the owning lane
      const uint32_t col = owner * COLS + c;                      // column offset inside the warp
      if (col < rows_here) {
        const uint8_t* src = area + r * kPitch + ch * 16;
        uint4 v;
        if (bits == 6) {
          const uint2 a = reinterpret_cast<const uint2*>(src)[0], b = reinterpret_cast<const uint2*>(src)[1];
          v = make_uint4(a.x, a.y, b.x, b.y);
        } else {
          v = *reinterpret_cast<const uint4*>(src);
        }
        uint8_t* g = elems + (size_t)(o * inner + warp_col0 + col) * out_row_bytes + (size_t)kb0 * kBpb + ch * 16;
        *reinterpret_cast<uint4*>(g) = v;
      }
    }
    __syncwarp();
  }
}

// ---------------------------------------------------------------------------
// Host-side dispatch
// ---------------------------------------------------------------------------

template <int FMT, int ROUND, int DTYPE, int LAYOUT, bool AL32>
static cudaError_t launch_lastaxis_al(const QuantizeArgs& a) {
  constexpr int U = kUnitsPerThread;
  constexpr int kElems = LastAxis<DTYPE>::kElems;
  const uint32_t n_units = (uint32_t)(a.numel / kElems);
  const uint32_t n_blocks = (uint32_t)(a.numel / kBlock);
  const uint32_t kblocks = (uint32_t)(a.L / kBlock);
  const uint32_t span = kThreads * U;
  auto kernel = quantize_lastaxis_kernel<FMT, ROUND, DTYPE, LAYOUT, AL32, U>;
  // one CTA per 256 units, no grid-stride loop: in steady state the block scheduler's natural
  // desynchronisation of CTAs beat a persistent grid by 5-10 %
  const uint32_t grid = (n_units + span - 1) / span;
  const FastDiv kd = make_fastdiv(kblocks);
  // one 32-bit store per four scale bytes when groups of four never straddle a row or the end
  const uint32_t scale_words = LAYOUT == MX_SCALES_LINEAR ? (n_blocks % 4 == 0) : (kblocks % 4 == 0);
  return launch_pdl(kernel, dim3(grid), dim3(kThreads), 0, a.stream, a.in, a.elems, a.scales, n_units, kblocks, kd,
                    scale_words);
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
  const uint32_t grid_x = (threads_x + kStridedThreads - 1) / kStridedThreads;
  // consecutive blocks of a column are written by the same thread (their codes are adjacent in
  // the output row); fewer per thread when the grid would otherwise not fill the machine
  // (an 8-bit block is a whole 32-byte sector by itself: one block per thread and CTA keeps the
  // CTAs short-lived and the end of the grid even -- 8192 x 28672 BF16 -> E4M3: 132 -> 109 us)
  const uint32_t kb_cap = FmtTraits<FMT>::bits == 8 ? 1u : 4u;
  uint32_t kb_per_thread = kblocks < kb_cap ? kblocks : kb_cap;
  const uint64_t outer_eff = a.outer < 65535 ? (uint64_t)a.outer : 65535;
  while (kb_per_thread > 1 &&
         (uint64_t)grid_x * ((kblocks + kb_per_thread - 1) / kb_per_thread) * outer_eff < (uint64_t)a.sm_count * 16)
    kb_per_thread >>= 1;
  dim3 grid(grid_x, (kblocks + kb_per_thread - 1) / kb_per_thread, (uint32_t)outer_eff);
  // FP32 input (8-byte loads of two columns): a grid that is resident all at once reads without L1 allocation
  if constexpr (DTYPE == MX_F32 && COLS == 2) {
    if ((uint64_t)grid.x * grid.y * grid.z <= 4ull * (uint64_t)a.sm_count)
      return launch_pdl(quantize_strided_kernel<FMT, ROUND, DTYPE, LAYOUT, COLS, true>, grid, dim3(kStridedThreads), 0,
                        a.stream, a.in, a.elems, a.scales, (uint32_t)a.outer, (uint32_t)a.L, (uint32_t)a.inner,
                        kb_per_thread);
  }
  return launch_pdl(quantize_strided_kernel<FMT, ROUND, DTYPE, LAYOUT, COLS>, grid, dim3(kStridedThreads), 0,
                    a.stream, a.in, a.elems, a.scales, (uint32_t)a.outer, (uint32_t)a.L, (uint32_t)a.inner,
                    kb_per_thread);
}

template <int FMT, int ROUND, int DTYPE, int LAYOUT>
static cudaError_t launch_strided(const QuantizeArgs& a) {
  // widest column group whose loads stay aligned: 8 bytes per row and thread
  constexpr int kWide = DTYPE == MX_BF16 ? 4 : 2;
  constexpr int bits = FmtTraits<FMT>::bits;
  const uint32_t kblocks = (uint32_t)(a.L / kBlock);
  const bool wide = a.inner % kWide == 0 && (uintptr_t)a.in % 8 == 0;
  // 6- and 4-bit codes go through the staged kernel (their per-lane stores would be partial
  // sectors); 8-bit codes are whole 32-byte sectors per lane already and are faster direct
  const bool staged = bits != 8 && wide && kblocks % 4 == 0 && (a.L * bits / 8) % 16 == 0 && (uintptr_t)a.elems % 16 == 0 &&
                      (uintptr_t)a.scales % 4 == 0;
  if (staged) {
    constexpr uint32_t NB = bits == 4 ? 2 : 4;  // blocks per CTA, as in the kernel
    constexpr uint32_t kPitch = NB * kBlock * bits / 8 + (bits == 6 ? 8 : 16);
    constexpr uint32_t smem = (kStagedThreads / 32) * 32 * kWide * kPitch;
    static_assert(smem <= 48 * 1024, "staging fits the default shared-memory limit");
    const uint32_t threads_x = (uint32_t)(a.inner / kWide);
    dim3 grid((threads_x + kStagedThreads - 1) / kStagedThreads, kblocks / NB,
              (uint32_t)(a.outer < 65535 ? a.outer : 65535));
    if constexpr (DTYPE == MX_F32) {  // (see ld_row8)
      if ((uint64_t)grid.x * grid.y * grid.z <= 8ull * (uint64_t)a.sm_count)
        return launch_pdl(quantize_strided_staged_kernel<FMT, ROUND, DTYPE, LAYOUT, kWide, true>, grid,
                          dim3(kStagedThreads), smem, a.stream, a.in, a.elems, a.scales, (uint32_t)a.outer,
                          (uint32_t)a.L, (uint32_t)a.inner);
    }
    return launch_pdl(quantize_strided_staged_kernel<FMT, ROUND, DTYPE, LAYOUT, kWide>, grid,
                      dim3(kStagedThreads), smem, a.stream, a.in, a.elems, a.scales, (uint32_t)a.outer,
                      (uint32_t)a.L, (uint32_t)a.inner);
  }
  if (wide) return launch_strided_cols<FMT, ROUND, DTYPE, LAYOUT, kWide>(a);
  return launch_strided_cols<FMT, ROUND, DTYPE, LAYOUT, 1>(a);
}

// ---------------------------------------------------------------------------
// Axis lengths that are not a multiple of 32
// ---------------------------------------------------------------------------

// The axis then ends in a partial block: its missing elements count as +0 (they cannot change the
// block maximum and encode as code 0) and the stored row is padded with zero codes to a whole
// block.  The same kernel writes rows zero-extended to a multiple of 128 elements when the caller asks
// for them (kblocks then counts the stored blocks; those past the axis end come out as zero codes
// under scale byte 0).  Rare shapes, so one plain kernel serves every layout: a thread converts one block of the
// [outer, L, inner] tensor, element by element; consecutive threads take consecutive inner
// positions (coalesced when the axis is strided) or consecutive blocks of a row.
template <int FMT, int ROUND, int DTYPE, int LAYOUT>
__global__ void __launch_bounds__(256)
quantize_tail_kernel(const void* __restrict__ in, uint8_t* __restrict__ elems, uint8_t* __restrict__ scales,
                     uint32_t outer, uint32_t L, uint32_t inner, uint32_t kblocks, uint64_t total_blocks) {
  constexpr int bits = FmtTraits<FMT>::bits;
  pdl_prologue();
  for (uint64_t b = (uint64_t)blockIdx.x * 256 + threadIdx.x; b < total_blocks; b += (uint64_t)gridDim.x * 256) {
    uint32_t o, kb, j;
    if (inner > 1) {
      j = (uint32_t)(b % inner);
      const uint64_t t = b / inner;
      kb = (uint32_t)(t % kblocks);
      o = (uint32_t)(t / kblocks);
    } else {
      j = 0;
      kb = (uint32_t)(b % kblocks);
      o = (uint32_t)(b / kblocks);
    }
    const uint32_t row = o * inner + j;
    float v[kBlock];
#pragma unroll
    for (int i = 0; i < kBlock; ++i) {
      const uint32_t k = kb * kBlock + i;
      float x = 0.0f;
      if (k < L) {
        const size_t idx = ((size_t)o * L + k) * inner + j;
        if (DTYPE == MX_BF16)
          x = __uint_as_float((uint32_t)__ldg(reinterpret_cast<const uint16_t*>(in) + idx) << 16);
        else
          x = __ldg(reinterpret_cast<const float*>(in) + idx);
      }
      v[i] = x;
    }
    float m = v[0];
#pragma unroll
    for (int i = 1; i < kBlock; ++i) m = absmax_nan(m, v[i]);
    const BlockScale s = block_scale<FMT>(m);
    uint32_t w[8];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      const float x[8] = {v[8 * g], v[8 * g + 1], v[8 * g + 2], v[8 * g + 3],
                          v[8 * g + 4], v[8 * g + 5], v[8 * g + 6], v[8 * g + 7]};
      cast8<FMT, ROUND>(x, s, w[2 * g], w[2 * g + 1]);
    }
    uint32_t* dst = reinterpret_cast<uint32_t*>(elems + (size_t)row * (kblocks * (kBlock * bits / 8)) +
                                                (size_t)kb * (kBlock * bits / 8));
    if (bits == 8) {
#pragma unroll
      for (int i = 0; i < 8; ++i) dst[i] = w[i];
    } else if (bits == 4) {
#pragma unroll
      for (int i = 0; i < 4; ++i) dst[i] = w[2 * i];
    } else {
      uint64_t q0, q1, q2;
      pack6(w, q0, q1, q2);
      dst[0] = (uint32_t)q0; dst[1] = (uint32_t)(q0 >> 32);
      dst[2] = (uint32_t)q1; dst[3] = (uint32_t)(q1 >> 32);
      dst[4] = (uint32_t)q2; dst[5] = (uint32_t)(q2 >> 32);
    }
    scales[scale_offset<LAYOUT>(row, kb, kblocks)] = (uint8_t)s.byte;
  }
}

template <int FMT, int ROUND, int DTYPE, int LAYOUT>
static cudaError_t launch_tail(const QuantizeArgs& a) {
  const uint32_t kblocks = (uint32_t)(a.L_store / kBlock);  // blocks past the axis end are all zero
  const uint64_t total = (uint64_t)a.outer * a.inner * kblocks;
  const uint64_t want = (total + 255) / 256, cap = (uint64_t)a.sm_count * 64;
  return launch_pdl(quantize_tail_kernel<FMT, ROUND, DTYPE, LAYOUT>, dim3((uint32_t)(want < cap ? want : cap)),
                    dim3(256), 0, a.stream, a.in, a.elems, a.scales, (uint32_t)a.outer, (uint32_t)a.L,
                    (uint32_t)a.inner, kblocks, total);
}

template <int FMT, int ROUND, int DTYPE, int LAYOUT>
static cudaError_t launch_any(const QuantizeArgs& a) {
  if (a.L % kBlock != 0 || a.L_store != a.L) return launch_tail<FMT, ROUND, DTYPE, LAYOUT>(a);
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
