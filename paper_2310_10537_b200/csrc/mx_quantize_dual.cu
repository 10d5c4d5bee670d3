// Fused dual-axis quantize: one read of a 2-D tensor X[R x C] produces both MX tensors a
// training step needs from it -- blocks along the rows' contiguous axis (the operand of X W)
// and blocks along the columns (the K-major [C x R] operand of X^T dY).  The paper's compute flow
// (Section 4.1) quantizes every matmul input in the forward and in the backward pass, and because
// quantizing and transposing do not commute (Section 3) the two are different tensors; reading X
// once instead of twice removes a third of that traffic.
//
// A warp owns a strip of 32*COLS columns (128 BF16 / 64 FP32) and walks four 32-row tiles:
//   column blocks  a thread holds 32 rows of its COLS columns packed in registers, exactly as the
//                  strided kernel does, and casts them; 8-bit codes go straight to the [C x R]
//                  output (one 32-byte sector per block), 6/4-bit codes are parked in shared
//                  memory and written as coalesced 96/64-byte runs after the four tiles;
//   row blocks     the same registers are written to a per-warp transpose area; lane r then reads
//                  row r of the tile (256 bytes = 4 BF16 / 2 FP32 blocks), casts those blocks and
//                  writes one contiguous 128/96/64 (BF16) or 64/48/32 (FP32) byte run of the
//                  [R x C] output.
// Only __syncwarp is needed: every warp has private shared-memory areas.
// Used for FP32 input (8- and 4-bit codes, and 6-bit codes of tensors that are not whole 128 x 128
// tiles); BF16 input and the other FP32 cases go through the tile kernels of mx_quantize_tile.cu.
#include "mx_device.cuh"
#include "mx_launch.h"
#include "mx_quantize_common.cuh"

namespace mx {

constexpr int kDualThreads = 64;
constexpr uint32_t kTPitch = 32 * 8 + 16;  // transpose area: 32 lanes x 8 bytes per tile row + pad

template <int FMT, int DTYPE> struct DualCfg {
  static constexpr int bits = FmtTraits<FMT>::bits;
  static constexpr int COLS = DTYPE == MX_BF16 ? 4 : 2;
  static constexpr uint32_t kBpb = kBlock * bits / 8;
  static constexpr uint32_t kSeg = 4 * kBpb;                         // four column blocks of one column
  static constexpr uint32_t kPitch = kSeg + (bits == 6 ? 8 : 16);
  static constexpr uint32_t kStageBytes = bits == 8 ? 0 : 32 * COLS * kPitch;  // per warp
  static constexpr uint32_t kWarpBytes = 32 * kTPitch + kStageBytes;
  static constexpr uint32_t kSmem = (kDualThreads / 32) * kWarpBytes;
};

// Resident CTAs per SM (CTAS): six for FP32 input (about 150 registers), except 8-bit codes on
// tensors of three waves or more, which gain 5 % at eight (128 registers).  The staged 6- and 4-bit
// variants cannot follow: seven or eight of their CTAs need more than 196 KB of shared memory, which
// leaves 28 KB of L1, and the loads in flight live there (69 -> 89 us on 8192 x 8192; the same
// happens to every variant when the largest shared-memory carve-out is forced).  One-wave tensors
// lose at eight too (4096 x 4096: 20.1 -> 21.6 us).  (The BF16 instances, four CTAs of 255
// registers, are no longer built: the tile kernels replaced them.)
template <int FMT, int ROUND, int DTYPE, int LAYOUT, int CTAS>
__global__ void __launch_bounds__(kDualThreads, CTAS)
quantize_dual_kernel(const void* __restrict__ in, uint8_t* __restrict__ elems_row,
                     uint8_t* __restrict__ scales_row, uint8_t* __restrict__ elems_col,
                     uint8_t* __restrict__ scales_col, uint32_t R, uint32_t C, uint32_t tiles_per_warp) {
  using cfg = DualCfg<FMT, DTYPE>;
  constexpr int bits = cfg::bits;
  constexpr int COLS = cfg::COLS;
  constexpr int kWords = StridedRow<DTYPE, COLS>::kWords;  // 2
  constexpr uint32_t kBpb = cfg::kBpb;
  constexpr int kRowBlocks = DTYPE == MX_BF16 ? 4 : 2;      // row blocks in a tile row of the strip
  extern __shared__ __align__(16) uint8_t dual_smem[];
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint8_t* tarea = dual_smem + warp * cfg::kWarpBytes;
  uint8_t* sarea = tarea + 32 * kTPitch;
  const uint32_t strip = blockIdx.x * (kDualThreads / 32) + warp;   // column strip of 32*COLS columns
  const uint32_t warp_col0 = strip * 32 * COLS;
  pdl_prologue();
  if (warp_col0 >= C) return;
  const uint32_t col0 = warp_col0 + lane * COLS;
  const size_t esz = DTYPE == MX_BF16 ? 2 : 4;
  const size_t in_pitch = (size_t)C * esz;
  const uint32_t kb_row = C / kBlock, kb_col = R / kBlock;          // blocks per output row
  const size_t row_out_bytes = (size_t)C * bits / 8, col_out_bytes = (size_t)R * bits / 8;
  // 32-row tiles this warp walks: four, or fewer when that fills the machine more evenly (the staged
  // 6- and 4-bit column codes: at least two, so that a row's run is 48 / 32 bytes)
  const uint32_t T = bits == 8 ? tiles_per_warp : max(tiles_per_warp, 2u);
  const uint32_t tile0 = blockIdx.y * T;                             // first 32-row tile of this CTA

  uint32_t col_scale_word[COLS];
#pragma unroll
  for (int c = 0; c < COLS; ++c) col_scale_word[c] = 0;

  // The 32 rows of a tile are loaded one tile ahead: the loads of tile j + 1 are issued as soon as
  // the column arithmetic has consumed the registers of tile j and fly during its row arithmetic.
  uint32_t raw[kBlock][kWords];
  auto load_tile = [&](uint32_t tile) {
    const char* p = reinterpret_cast<const char*>(in) + (size_t)tile * kBlock * in_pitch + (size_t)col0 * esz;
#pragma unroll
    for (int k = 0; k < kBlock; ++k) {
      const uint2 w = ld_cg8(p + (size_t)k * in_pitch);
      raw[k][0] = w.x; raw[k][1] = w.y;
    }
  };
  load_tile(tile0);

#pragma unroll 1
  for (uint32_t j = 0; j < T; ++j) {
    const uint32_t tile = tile0 + j;
    // transpose area first, so the shared-memory latency hides behind the column arithmetic
#pragma unroll
    for (int k = 0; k < kBlock; ++k)
      *reinterpret_cast<uint2*>(tarea + k * kTPitch + lane * 8) = make_uint2(raw[k][0], raw[k][1]);

    // ---- column blocks: (column col0 + c, rows of this tile) -> output row col0 + c, block `tile`
    float amax[COLS];
    column_amax<DTYPE, COLS>(raw, amax);
#pragma unroll
    for (int c = 0; c < COLS; ++c) {
      const BlockScale s = block_scale<FMT>(amax[c]);
      col_scale_word[c] |= s.byte << (8 * j);
      uint32_t w[8];
      column_cast<FMT, ROUND, DTYPE, COLS>(raw, c, s, w);
      if (bits == 8) {
        uint8_t* dst = elems_col + (size_t)(col0 + c) * col_out_bytes + (size_t)tile * kBpb;
        store_run<8>(dst, w, (reinterpret_cast<uintptr_t>(dst) & 31u) == 0);
      } else {
        uint8_t* dst = sarea + (c * 32 + lane) * cfg::kPitch + j * kBpb;
        if (bits == 4) {
          reinterpret_cast<uint4*>(dst)[0] = make_uint4(w[0], w[2], w[4], w[6]);
        } else {
          uint64_t q0, q1, q2;
          pack6(w, q0, q1, q2);
          uint2* d2 = reinterpret_cast<uint2*>(dst);
          d2[0] = make_uint2((uint32_t)q0, (uint32_t)(q0 >> 32));
          d2[1] = make_uint2((uint32_t)q1, (uint32_t)(q1 >> 32));
          d2[2] = make_uint2((uint32_t)q2, (uint32_t)(q2 >> 32));
        }
      }
    }
    __syncwarp();
    if (j + 1 < T) load_tile(tile + 1);

    // ---- row blocks: lane r owns row (tile * 32 + r) of the strip: kRowBlocks blocks of 32 columns
    {
      const uint32_t row = tile * kBlock + lane;
      const uint8_t* src = tarea + lane * kTPitch;
      uint32_t codes[kRowBlocks][8];
      uint32_t row_scale_word = 0;
#pragma unroll
      for (int q = 0; q < kRowBlocks; ++q) {
        // a block is 64 bytes (BF16) or 128 bytes (FP32) of the row
        constexpr int kUnits = DTYPE == MX_BF16 ? 1 : 2;
        uint32_t u[kUnits][16];
#pragma unroll
        for (int h = 0; h < kUnits; ++h)
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint4 v = *reinterpret_cast<const uint4*>(src + (q * kUnits + h) * 64 + i * 16);
            u[h][4 * i] = v.x; u[h][4 * i + 1] = v.y; u[h][4 * i + 2] = v.z; u[h][4 * i + 3] = v.w;
          }
        float am = unit_amax<DTYPE>(u[0]);
        if (kUnits == 2) am = absmax_nan(am, unit_amax<DTYPE>(u[kUnits - 1]));
        const BlockScale s = block_scale<FMT>(am);
        row_scale_word |= s.byte << (8 * q);
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          float x[8];
          if (DTYPE == MX_BF16) unit_group<DTYPE>(u[0], g, x);
          else unit_group<DTYPE>(u[(g / 2) % kUnits], g % 2, x);
          cast8<FMT, ROUND>(x, s, codes[q][2 * g], codes[q][2 * g + 1]);
        }
      }
      // contiguous run of kRowBlocks blocks in the [R x C] output
      uint8_t* dst = elems_row + (size_t)row * row_out_bytes + (size_t)strip * kRowBlocks * kBpb;
      const bool wide = (reinterpret_cast<uintptr_t>(dst) & 31u) == 0;
      if (bits == 8) {
        uint32_t run[kRowBlocks * 8];
#pragma unroll
        for (int q = 0; q < kRowBlocks; ++q)
#pragma unroll
          for (int i = 0; i < 8; ++i) run[8 * q + i] = codes[q][i];
        store_run<kRowBlocks * 8>(dst, run, wide);
      } else if (bits == 4) {
        uint32_t run[kRowBlocks * 4];
#pragma unroll
        for (int q = 0; q < kRowBlocks; ++q)
#pragma unroll
          for (int i = 0; i < 4; ++i) run[4 * q + i] = codes[q][2 * i];
        store_run<kRowBlocks * 4>(dst, run, wide);
      } else {
        uint32_t run[kRowBlocks * 6];
#pragma unroll
        for (int q = 0; q < kRowBlocks; ++q) {
          uint64_t a, b, c;
          pack6(codes[q], a, b, c);
          run[6 * q] = (uint32_t)a; run[6 * q + 1] = (uint32_t)(a >> 32);
          run[6 * q + 2] = (uint32_t)b; run[6 * q + 3] = (uint32_t)(b >> 32);
          run[6 * q + 4] = (uint32_t)c; run[6 * q + 5] = (uint32_t)(c >> 32);
        }
        store_run<kRowBlocks * 6>(dst, run, wide);
      }
      uint8_t* sdst = scales_row + scale_offset<LAYOUT>(row, strip * kRowBlocks, kb_row);
      if (kRowBlocks == 4) *reinterpret_cast<uint32_t*>(sdst) = row_scale_word;
      else *reinterpret_cast<uint16_t*>(sdst) = (uint16_t)row_scale_word;
    }
    __syncwarp();  // the transpose area is rewritten by the next tile
  }

  // ---- column outputs of the four tiles
#pragma unroll
  for (int c = 0; c < COLS; ++c)
  {
    uint8_t* sp = scales_col + scale_offset<LAYOUT>(col0 + c, tile0, kb_col);  // T adjacent bytes, T-aligned
    if (T == 4) *reinterpret_cast<uint32_t*>(sp) = col_scale_word[c];
    else if (T == 2) *reinterpret_cast<uint16_t*>(sp) = (uint16_t)col_scale_word[c];
    else *sp = (uint8_t)col_scale_word[c];
  }
  if (bits != 8) {
    __syncwarp();
    // every output row's run of T blocks, consecutive lanes on consecutive chunks: 32-byte chunks
    // (whole sectors per request) where the run and the tensor allow, else 16-byte ones
    const uint32_t seg = T * kBpb;
    const bool wide = ((reinterpret_cast<uintptr_t>(elems_col) | col_out_bytes) & 31u) == 0 && seg % 32 == 0;
    const uint32_t cb = wide ? 32u : 16u, nch = seg / cb;
    for (uint32_t i = lane; i < 32 * COLS * nch; i += 32) {
      const uint32_t r = i / nch, ch = i - r * nch;
      const uint32_t c = r >> 5, owner = r & 31;
      const uint2* src = reinterpret_cast<const uint2*>(sarea + r * cfg::kPitch + ch * cb);
      uint8_t* g = elems_col + (size_t)(warp_col0 + owner * COLS + c) * col_out_bytes + (size_t)tile0 * kBpb + ch * cb;
      const uint2 q0 = src[0], q1 = src[1];
      if (wide) {
        const uint2 q2 = src[2], q3 = src[3];
        const uint32_t v[8] = {q0.x, q0.y, q1.x, q1.y, q2.x, q2.y, q3.x, q3.y};
        st_32(g, v);
      } else {
        *reinterpret_cast<uint4*>(g) = make_uint4(q0.x, q0.y, q1.x, q1.y);
      }
    }
  }
}

template <int FMT, int ROUND, int DTYPE, int LAYOUT, int CTAS>
static cudaError_t launch_dual_ctas(const DualArgs& a) {
  using cfg = DualCfg<FMT, DTYPE>;
  static_assert(cfg::kSmem <= 48 * 1024, "fits the default shared-memory limit");
  const uint32_t strips = (uint32_t)(a.C / (32 * cfg::COLS));
  const uint32_t ctas_x = (strips + kDualThreads / 32 - 1) / (kDualThreads / 32);
  // Tiles per warp: the choice that needs the least time in units of one tile, given
  // how many warps are resident at once -- e.g. 4096 x 4096 FP32 is 1.15 waves of four-tile warps
  // (two rounds) but 4.6 waves of one-tile warps (five rounds of a quarter the length).
  uint32_t T = 4;
  {
    const uint64_t slots = (uint64_t)a.sm_count * CTAS;  // resident CTAs
    uint64_t best = ~0ull;
    for (uint32_t t : {4u, 2u, 1u}) {
      if (t == 1 && cfg::bits != 8) continue;
      const uint64_t ctas = (uint64_t)ctas_x * (uint64_t)(a.R / 32 / t);
      // in units of a fifth of a tile; two-tile warps of 6-bit codes write 48-byte runs as half
      // sectors, which measured about a fifth slower per tile
      const uint64_t cost = (ctas + slots - 1) / slots * t * ((cfg::bits == 6 && t == 2) ? 6 : 5);
      if (cost < best) { best = cost; T = t; }
    }
  }
  dim3 grid(ctas_x, (uint32_t)(a.R / 32 / T));
  auto kernel = quantize_dual_kernel<FMT, ROUND, DTYPE, LAYOUT, CTAS>;
  return launch_pdl(kernel, grid, dim3(kDualThreads), cfg::kSmem,
                    a.stream, a.in, a.elems_row, a.scales_row, a.elems_col, a.scales_col, (uint32_t)a.R,
                    (uint32_t)a.C, T);
}

template <int FMT, int ROUND, int DTYPE, int LAYOUT>
static cudaError_t launch_dual_t(const DualArgs& a) {
  if constexpr (DTYPE == MX_BF16) {
    return launch_dual_ctas<FMT, ROUND, DTYPE, LAYOUT, 4>(a);
  } else {
    if constexpr (FmtTraits<FMT>::bits == 8) {
      // four-tile warps of the whole tensor against the warps resident at eight CTAs per SM
      const uint64_t warps = (uint64_t)(a.C / 64) * (uint64_t)(a.R / 128);
      if (warps >= 3ull * 16ull * (uint64_t)a.sm_count) return launch_dual_ctas<FMT, ROUND, DTYPE, LAYOUT, 8>(a);
    }
    return launch_dual_ctas<FMT, ROUND, DTYPE, LAYOUT, 6>(a);
  }
}

// FP32 input only: BF16 tensors go through the tile kernels (mx_quantize_tile.cu), which replaced
// this kernel's BF16 instances (255 registers, 8 warps per SM).
template <int FMT, int ROUND>
static cudaError_t dispatch_dual(const DualArgs& a) {
  if (a.dtype != MX_F32) return cudaErrorInvalidValue;
  return a.layout == MX_SCALES_LINEAR ? launch_dual_t<FMT, ROUND, MX_F32, MX_SCALES_LINEAR>(a)
                                      : launch_dual_t<FMT, ROUND, MX_F32, MX_SCALES_SWIZZLED>(a);
}

template <int FMT>
static cudaError_t dispatch_dual_round(const DualArgs& a) {
  return a.rounding == MX_RHAZ ? dispatch_dual<FMT, MX_RHAZ>(a) : dispatch_dual<FMT, MX_RNE>(a);
}

cudaError_t launch_quantize_dual(const DualArgs& a) {
  switch (a.fmt) {
    case MX_E4M3: return dispatch_dual_round<MX_E4M3>(a);
    case MX_E5M2: return dispatch_dual_round<MX_E5M2>(a);
    case MX_E3M2: return dispatch_dual_round<MX_E3M2>(a);
    case MX_E2M3: return dispatch_dual_round<MX_E2M3>(a);
    case MX_E2M1: return dispatch_dual_round<MX_E2M1>(a);
    default: return dispatch_dual_round<MX_INT8>(a);
  }
}

}  // namespace mx
