// Quantize of a BF16 tensor through shared-memory tiles: X[R x C] is read once, by TMA, in tiles of
// 128 rows x 128 columns, and each tile is quantized out of shared memory along its rows (blocks
// along the contiguous axis: the operand of X W) and along its columns (blocks along axis 0: the
// K-major [C x R] operand of X^T dY).  The paper's compute flow (Section 4.1) quantizes every matmul
// input in the forward and in the backward pass, and because quantizing and transposing do not
// commute (Section 3) those are two tensors; producing both from one read removes a third of the
// traffic.
//
// Why through shared memory: a thread that keeps 32 rows of a block in registers (the kernel in
// mx_quantize_dual.cu, used for FP32 input) needs ~250 registers once BF16 packs twice the
// elements into them and both directions are served, which leaves eight warps per SM -- too few
// loads in flight to cover HBM latency (measured: 11 % of the warp slots active, DRAM 47 % busy).
// Here the copies in flight cost no registers: a CTA keeps tiles (32 KB each, two TMA boxes of 128
// rows x 128 bytes in the 128-byte swizzle) on their way while it converts one, two CTAs share an
// SM, and a converting thread holds one block at a time.  The swizzle makes both access directions
// conflict-free: a row's 16-byte chunks are spread over the banks by (chunk ^ row % 8), a word
// column's 32 lanes always hit 32 different banks.  Every mbarrier wait is bounded: when one runs
// out the CTA records it in a status word and leaves.
//
// The kernels (no meeting of warps in any of them: every warp writes whole 32-byte sectors by
// itself -- sub-byte codes: lanes exchange part sectors by shuffle --, a producer warp refills a
// stage when its readers have released it, tiles are dealt out at run time):
//   quantize_tile_dual_kernel      BF16 input, every format, both outputs (mx_quantize_dual).
//                                  8192 x 8192: E4M3 46.8 us, E3M2 44.0, E2M1 34.5 (0.89 / 0.83 /
//                                  0.91 of the copy bandwidth on in + 2 x out bytes).  With its
//                                  Without its row pass it also serves mx_quantize along axis 0 for
//                                  6- and 4-bit codes (whole-tile tensors; 4096 x 16384: 30.2 us
//                                  against 35 for the 6-bit register kernel, 28.2 against 29.2 for 4-bit).
//   quantize_tile_dual_f32_kernel  FP32 input, 6-bit codes, both outputs: 8192 x 8192 in 56.9 us
//                                  (the copy bandwidth).
// (A first tile kernel -- 256 threads, warps 0-3 rows, warps 4-7 columns with the sub-byte codes
// parked in shared memory, a CTA barrier per tile, tiles split evenly -- measured 53 / 47 / 41 us
// on 8192 x 8192 BF16 for E4M3 / E3M2 / E2M1 and 32.3 us in its column-only form on 4096 x 16384;
// timing-only builds of it: copies alone 22 us, both passes without their stores 33, one pass with
// its stores 35.)
#include <atomic>

#include "mx_device.cuh"
#include "mx_launch.h"
#include "mx_quantize_common.cuh"
#include "mx_tmap.h"

namespace mx {

namespace {

constexpr uint32_t kTileRows = 128;
constexpr uint32_t kBoxBytes = kTileRows * 128;   // one TMA box: 128 rows x 128 bytes
constexpr long long kTileSpinLimit = 2000000000LL;

__device__ unsigned int g_tile_status;  // 1: a tile never arrived (bounded wait ran out)

// Tile counters of the kernels that deal their tiles out at run time: a launch takes one slot of
// two words -- [0] tiles handed out beyond every CTA's first, [1] CTAs that have finished -- and
// leaves both at zero: the CTA that finishes last resets the slot (no CTA asks for a tile after it
// has been told that there are none left, and it is counted as finished only after that).  The host
// cycles through the slots, so that launches in flight on different streams do not share one.
constexpr uint32_t kSchedSlots = 256;
__device__ unsigned int g_tile_sched[2 * kSchedSlots];
inline uint32_t next_sched_slot() {
  static std::atomic<uint32_t> next{0};
  return next.fetch_add(1, std::memory_order_relaxed) % kSchedSlots;
}

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar) : "memory");
}

__device__ __forceinline__ bool tile_wait(uint32_t bar, uint32_t parity) {
  auto try_wait = [&]() {
    uint32_t ok;
    asm volatile(
        "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
  };
  if (try_wait()) return true;
  const long long t0 = clock64();
  for (uint32_t it = 1;; ++it) {
    if (try_wait()) return true;
    if ((it & 63u) == 0 && clock64() - t0 > kTileSpinLimit) return false;
  }
}

// 16-byte chunk c (0..7) of row r of a box, as the 128-byte swizzle stores it.
__device__ __forceinline__ uint32_t box_chunk(uint32_t box_base, uint32_t r, uint32_t c) {
  return box_base + r * 128u + ((c ^ (r & 7u)) << 4);
}

// The producer warp of the kernels below.  Tiles are dealt out at run time: an SM's share of the
// memory system's bandwidth varies (with 128 x 256 tiles split evenly, 14 per CTA, the slowest of
// 147 CTAs took 95 k cycles and the median 79 k: 8192 x 8192 BF16 -> E4M3 in 51.3 us; dealt out, 47.0),
// so a CTA's first tile is its own index and every further one comes from the launch's counter.  The
// tile a stage holds is written beside the barriers before the stage is armed; a number past the
// last tile tells the readers to stop.  Barriers: "stage s has landed" at bar0 + 8 s, "stage s has
// been read" at bar0 + 8 (STAGES + s); tile numbers at tile_id0 + 4 s.  A tile is BOXES boxes of 128
// rows x 128 bytes (box_cols elements) side by side.
template <uint32_t STAGES, uint32_t BOXES>
__device__ __forceinline__ void tile_producer(const CUtensorMap* tmap, uint32_t base, uint32_t bar0, uint32_t tile_id0,
                                              uint32_t box_cols, uint32_t tiles_c, uint32_t num_tiles,
                                              uint32_t sched_slot, uint32_t lane) {
  constexpr uint32_t kBytes = BOXES * kBoxBytes;
  unsigned int* sched = g_tile_sched + 2 * sched_slot;
  for (uint32_t it = 0;; ++it) {
    const uint32_t stage = it % STAGES, use = it / STAGES;
    if (use > 0 && !tile_wait(bar0 + 8 * (STAGES + stage), (use - 1) & 1u)) {  // its readers of the round before
      if (lane == 0) atomicCAS(&g_tile_status, 0u, 2u);
      break;
    }
    uint32_t t = blockIdx.x;
    if (it > 0) {
      if (lane == 0) t = gridDim.x + atomicAdd(&sched[0], 1u);
      t = __shfl_sync(0xFFFFFFFFu, t, 0);
    }
    if (lane == 0) {
      const uint32_t bar = bar0 + 8 * stage;
      asm volatile("st.shared.u32 [%0], %1;" ::"r"(tile_id0 + 4 * stage), "r"(t) : "memory");
      if (t < num_tiles) {
        const uint32_t tr = t / tiles_c, tc = t - tr * tiles_c;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(kBytes) : "memory");
        const uint32_t dst = base + stage * kBytes;
        for (uint32_t b = 0; b < BOXES; ++b)
          tma_load_2d(dst + b * kBoxBytes, tmap, (int)((tc * BOXES + b) * box_cols), (int)(tr * kTileRows), bar);
      } else {
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");  // nothing will land: complete the phase
      }
    }
    __syncwarp();
    if (t >= num_tiles) break;
  }
  // this CTA asks for no more tiles: count it; the last one leaves the slot as it found it
  if (lane == 0) {
    __threadfence();
    if (atomicInc(&sched[1], gridDim.x - 1u) == gridDim.x - 1u) atomicExch(&sched[0], 0u);
  }
}

// ---------------------------------------------------------------------------------------------
// Both passes, no meeting of warps.  Nothing is gathered across warps before it is written: every
// warp converts its share of a tile straight out of the (read-only) stage and writes whole 32-byte
// sectors by itself, and the only synchronisation left is the stage's two barriers -- "tile landed"
// (the copy engine) and "tile read" (one arrival per warp), which a producer warp waits on before
// it refills the stage.  A block of 8-bit codes is a sector; two blocks of 4-bit codes are, and
// four blocks of 6-bit codes are three, so for those two or four lanes pass words to each other
// (see the 4- and 6-bit branches).  The lane maps of 8- and 4-bit codes:
// With NBOX boxes of 64 columns side by side in a tile (NBOX x 128 contiguous bytes of every row):
//   warps 0 .. 4 NBOX - 1
//               row pass: lane (r, h) = (lane % (32 / NBOX), lane / (32 / NBOX)) converts the two
//               blocks that row (32 / NBOX) w + r has in box h (one 128-byte box row: eight 16-byte
//               loads; a quarter-warp reads eight rows of one box, conflict-free under the
//               128-byte swizzle) and writes them as one 64-byte run plus two adjacent scale bytes;
//               column pass: warp w = (box b, row group g) = (w % NBOX, w / NBOX), lane = one 32-bit
//               word column of box b (two columns), 32 rows down (32 conflict-free 4-byte loads):
//               two whole-sector stores and two scale bytes
//   warp 4 NBOX producer: one lane issues the box copies of a tile into a stage once its readers
//               have released it
// ---------------------------------------------------------------------------------------------
// Two boxes: tiles of 128 x 128, eight reader warps + the producer, three stages of 32 KB, two
// CTAs per SM.  Measured with the tiles dealt out at run time (see the producer): 46.9 us on 8192 x
// 8192 and 15.7 on 4096 x 4096, against 47.2 and 16.4 with four boxes (128 x 256 tiles, 16 reader
// warps, one CTA per SM); with a static split of the tiles it was the other way round (52.8 / 51.3).
constexpr uint32_t kTdBoxes = 2;
constexpr uint32_t kTdWarps = 4 * kTdBoxes;
constexpr int kTileDualThreads = 32 * (kTdWarps + 1);
constexpr uint32_t kTdTileBytes = kTdBoxes * kBoxBytes;
constexpr uint32_t kTdCols = 64 * kTdBoxes;
constexpr int kTdCtasPerSm = kTdBoxes == 2 ? 2 : 1;

template <int FMT, int ROUND, int LAYOUT, bool COLS_ONLY = false>
__global__ void __launch_bounds__(kTileDualThreads, kTdCtasPerSm)
quantize_tile_dual_kernel(const __grid_constant__ CUtensorMap tmap_in, uint8_t* __restrict__ elems_row,
                      uint8_t* __restrict__ scales_row, uint8_t* __restrict__ elems_col,
                      uint8_t* __restrict__ scales_col, uint32_t R, uint32_t C, uint32_t tiles_c,
                      uint32_t num_tiles, uint32_t sched_slot) {
  constexpr int bits = FmtTraits<FMT>::bits;
  static_assert(bits == 8 || kTdBoxes == 2, "sub-byte codes: 128 x 128 tiles (their lane maps assume two boxes)");
  constexpr int DTYPE = MX_BF16;
  constexpr uint32_t kStages = 3;
  constexpr uint32_t kWarps = kTdWarps;  // reader warps
  constexpr uint32_t kBpb = kBlock * bits / 8;  // 32 or 16 bytes of codes per block
  extern __shared__ uint8_t tile_smem_raw[];
  const uint32_t base = (smem_addr(tile_smem_raw) + 1023u) & ~1023u;
  const uint32_t bar0 = base + kStages * kTdTileBytes;      // full[s] at 8 s, empty[s] at 8 (kStages + s)
  const uint32_t tile_id0 = bar0 + 16 * kStages;            // the tile a stage holds (written by the producer)
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    for (uint32_t s = 0; s < kStages; ++s) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar0 + 8 * s) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar0 + 8 * (kStages + s)), "r"(kWarps) : "memory");
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_in)) : "memory");
  }
  __syncthreads();
  pdl_prologue();
  const uint32_t kb_row = C / kBlock, kb_col = R / kBlock;
  const size_t row_out_bytes = (size_t)kb_row * kBpb, col_out_bytes = (size_t)kb_col * kBpb;

  if (warp == kWarps) {
    tile_producer<kStages, kTdBoxes>(&tmap_in, base, bar0, tile_id0, 64u, tiles_c, num_tiles, sched_slot, lane);
    return;
  }

  // -------------------------------- readers --------------------------------
#pragma unroll 1
  for (uint32_t it = 0;; ++it) {
    const uint32_t stage = it % kStages, parity = (it / kStages) & 1u;
    if (!tile_wait(bar0 + 8 * stage, parity)) {
      if (lane == 0) atomicCAS(&g_tile_status, 0u, 1u);
      return;
    }
    uint32_t t;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(t) : "r"(tile_id0 + 4 * stage) : "memory");
    if (t >= num_tiles) return;  // no tile left
    const uint32_t tr = t / tiles_c, tc = t - tr * tiles_c;
    const uint32_t tile_base = base + stage * kTdTileBytes;
    const uint32_t row0 = tr * kTileRows, col0 = tc * kTdCols;
    if constexpr (bits != 6 && !COLS_ONLY) {  // row pass: the two blocks of one row that lie in one box; a quarter-warp = 8 consecutive rows of a box
      constexpr uint32_t kRowsPerWarp = 32 / kTdBoxes;   // 16 or 8
      const uint32_t r = warp * kRowsPerWarp + (lane % kRowsPerWarp), h = lane / kRowsPerWarp;
      const uint32_t box = tile_base + h * kBoxBytes;
      uint32_t codes[2][8];
      uint32_t scale_pair = 0;
#pragma unroll
      for (uint32_t q = 0; q < 2; ++q) {
        uint32_t u[16];
#pragma unroll
        for (uint32_t i = 0; i < 4; ++i) {
          uint32_t v0, v1, v2, v3;
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                       : "=r"(v0), "=r"(v1), "=r"(v2), "=r"(v3) : "r"(box_chunk(box, r, q * 4u + i)));
          u[4 * i] = v0; u[4 * i + 1] = v1; u[4 * i + 2] = v2; u[4 * i + 3] = v3;
        }
        const BlockScale s = block_scale<FMT>(unit_amax<DTYPE>(u));
        scale_pair |= s.byte << (8 * q);
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          float x[8];
          unit_group<DTYPE>(u, g, x);
          cast8<FMT, ROUND>(x, s, codes[q][2 * g], codes[q][2 * g + 1]);
        }
      }
      const uint32_t row = row0 + r, kb0 = tc * (kTdCols / kBlock) + 2u * h;
      uint8_t* dst = elems_row + (size_t)row * row_out_bytes + (size_t)kb0 * kBpb;
      if (bits == 8) {
        const uint32_t run[16] = {codes[0][0], codes[0][1], codes[0][2], codes[0][3], codes[0][4], codes[0][5],
                                  codes[0][6], codes[0][7], codes[1][0], codes[1][1], codes[1][2], codes[1][3],
                                  codes[1][4], codes[1][5], codes[1][6], codes[1][7]};
        store_run<16>(dst, run, (reinterpret_cast<uintptr_t>(dst) & 31u) == 0);
      } else if (bits == 4) {  // a block is four words (cast8 leaves them in the even positions), two blocks one sector
        const uint32_t run[8] = {codes[0][0], codes[0][2], codes[0][4], codes[0][6],
                                 codes[1][0], codes[1][2], codes[1][4], codes[1][6]};
        store_run<8>(dst, run, (reinterpret_cast<uintptr_t>(dst) & 31u) == 0);
      }
      // two adjacent bytes in either layout (kb0 even, C % 128 == 0)
      *reinterpret_cast<uint16_t*>(scales_row + scale_offset<LAYOUT>(row, kb0, kb_row)) = (uint16_t)scale_pair;
    }
    if constexpr (bits == 8) {  // column pass: one word column (two columns) of one box, one 32-row group
      const uint32_t b = warp % kTdBoxes, g = warp / kTdBoxes;
      const uint32_t box = tile_base + b * kBoxBytes;
      const uint32_t c = lane >> 2, wofs = (lane & 3u) * 4u;
      uint32_t raw[kBlock][1];
#pragma unroll
      for (uint32_t k = 0; k < kBlock; ++k)
        asm volatile("ld.shared.b32 %0, [%1];" : "=r"(raw[k][0]) : "r"(box_chunk(box, g * kBlock + k, c) + wofs));
      float amax[2];
      column_amax<DTYPE, 2>(raw, amax);
      const uint32_t kb = tr * 4u + g;
#pragma unroll
      for (int cc = 0; cc < 2; ++cc) {
        const uint32_t col = col0 + b * 64u + lane * 2u + cc;
        const BlockScale s = block_scale<FMT>(amax[cc]);
        uint32_t cw[8];
        column_cast<FMT, ROUND, DTYPE, 2>(raw, cc, s, cw);
        uint8_t* dst = elems_col + (size_t)col * col_out_bytes + (size_t)kb * kBpb;
        store_run<8>(dst, cw, (reinterpret_cast<uintptr_t>(dst) & 31u) == 0);
        scales_col[scale_offset<LAYOUT>(col, kb, kb_col)] = (uint8_t)s.byte;
      }
    }
    if constexpr (bits == 4) {
      // column pass, 4-bit codes: a block is 16 bytes, so two lanes -- the same word column, row groups
      // 2 gp and 2 gp + 1 -- make up the 32-byte sector of each of their two columns: each keeps one
      // column and hands the other column's block (and scale byte) to its partner.  Warp w = (quarter
      // wq of the tile's 64 word columns, pair of row groups gp) = (w % 4, w / 4); lane = (word
      // column lane % 16, row group 2 gp + lane / 16).  (16 lanes read half a 128-byte row: a load
      // instruction touches two rows, two wavefronts.)
      const uint32_t wq = warp % 4u, gp = warp / 4u, hi = lane >> 4, g = 2u * gp + hi;
      const uint32_t w = 16u * (wq & 1u) + (lane & 15u);          // word column inside the box
      const uint32_t box = tile_base + (wq >> 1) * kBoxBytes;
      const uint32_t c = w >> 2, wofs = (w & 3u) * 4u;
      uint32_t raw[kBlock][1];
#pragma unroll
      for (uint32_t k = 0; k < kBlock; ++k)
        asm volatile("ld.shared.b32 %0, [%1];" : "=r"(raw[k][0]) : "r"(box_chunk(box, g * kBlock + k, c) + wofs));
      float amax[2];
      column_amax<DTYPE, 2>(raw, amax);
      uint32_t blk[2][4], sbyte[2];
#pragma unroll
      for (int cc = 0; cc < 2; ++cc) {
        const BlockScale s = block_scale<FMT>(amax[cc]);
        uint32_t cw[8];
        column_cast<FMT, ROUND, DTYPE, 2>(raw, cc, s, cw);
        sbyte[cc] = s.byte;
#pragma unroll
        for (int i = 0; i < 4; ++i) blk[cc][i] = cw[2 * i];
      }
      // keep column `hi`, give away column 1 - hi
      uint32_t mine[4], theirs[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        mine[i] = hi ? blk[1][i] : blk[0][i];
        theirs[i] = __shfl_xor_sync(0xFFFFFFFFu, hi ? blk[0][i] : blk[1][i], 16);
      }
      const uint32_t their_scale = __shfl_xor_sync(0xFFFFFFFFu, hi ? sbyte[0] : sbyte[1], 16);
      const uint32_t my_scale = hi ? sbyte[1] : sbyte[0];
      // blocks in order of their row groups: the even group's first
      const uint32_t run[8] = {hi ? theirs[0] : mine[0], hi ? theirs[1] : mine[1], hi ? theirs[2] : mine[2],
                               hi ? theirs[3] : mine[3], hi ? mine[0] : theirs[0], hi ? mine[1] : theirs[1],
                               hi ? mine[2] : theirs[2], hi ? mine[3] : theirs[3]};
      const uint32_t col = col0 + (wq >> 1) * 64u + w * 2u + hi;
      const uint32_t kb = tr * 4u + 2u * gp;
      uint8_t* dst = elems_col + (size_t)col * col_out_bytes + (size_t)kb * kBpb;
      store_run<8>(dst, run, (reinterpret_cast<uintptr_t>(dst) & 31u) == 0);
      const uint32_t pair = hi ? (their_scale | (my_scale << 8)) : (my_scale | (their_scale << 8));
      // two adjacent bytes in either layout (kb even)
      *reinterpret_cast<uint16_t*>(scales_col + scale_offset<LAYOUT>(col, kb, kb_col)) = (uint16_t)pair;
    }
    if constexpr (bits == 6) {
      // 6-bit codes: a block is 24 bytes, four blocks three sectors, so whole sectors need all four
      // blocks of a tile row or of a tile column in one place.  The warps split the roles: warps 4-7
      // convert rows (lane = one tile row: its four blocks, one 96-byte run), warps 0-3 columns --
      // warp w the w-th quarter of the tile's 64 word columns, in two steps of two row groups each
      // (lane = (word column lane % 16, row group 2 step + lane / 16): a load instruction touches two
      // rows, two wavefronts); the two lanes of a word column then hold row groups {0, 2} and {1, 3}
      // of both columns and pass eight words to each other so that one writes sectors 0 and 1 of
      // each column and the other sector 2.  Both roles convert 128 elements per lane and tile.
      if (warp >= 4u) {
        if constexpr (!COLS_ONLY) {
        const uint32_t r = (warp - 4u) * 32u + lane;
        uint32_t run[24];
        uint32_t scale_word = 0;
#pragma unroll
        for (uint32_t q = 0; q < 4; ++q) {
          const uint32_t box = tile_base + (q >> 1) * kBoxBytes;
          uint32_t u[16];
#pragma unroll
          for (uint32_t i = 0; i < 4; ++i) {
            uint32_t v0, v1, v2, v3;
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(v0), "=r"(v1), "=r"(v2), "=r"(v3) : "r"(box_chunk(box, r, (q & 1u) * 4u + i)));
            u[4 * i] = v0; u[4 * i + 1] = v1; u[4 * i + 2] = v2; u[4 * i + 3] = v3;
          }
          const BlockScale s = block_scale<FMT>(unit_amax<DTYPE>(u));
          scale_word |= s.byte << (8 * q);
          uint32_t cw[8], o[6];
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            float x[8];
            unit_group<DTYPE>(u, g, x);
            cast8<FMT, ROUND>(x, s, cw[2 * g], cw[2 * g + 1]);
          }
          pack6_words(cw, o);
#pragma unroll
          for (int i = 0; i < 6; ++i) run[6 * q + i] = o[i];
        }
        const uint32_t row = row0 + r, kb0 = tc * 4u;
        uint8_t* dst = elems_row + (size_t)row * row_out_bytes + (size_t)kb0 * kBpb;
        store_run<24>(dst, run, (reinterpret_cast<uintptr_t>(dst) & 31u) == 0);
        // four adjacent bytes in either layout (kb0 % 4 == 0)
        *reinterpret_cast<uint32_t*>(scales_row + scale_offset<LAYOUT>(row, kb0, kb_row)) = scale_word;
        }  // (COLS_ONLY: these warps only take part in the stage's barriers)
      } else {
        const uint32_t hi = lane >> 4;
        const uint32_t w = 16u * (warp & 1u) + (lane & 15u);        // word column inside the box
        const uint32_t box = tile_base + (warp >> 1) * kBoxBytes;
        const uint32_t c = w >> 2, wofs = (w & 3u) * 4u;
        uint32_t o[2][2][6];   // [step][column][word]: row group 2 step + hi
        uint32_t sb[2] = {0u, 0u};  // per column: this lane's two scale bytes at their positions in the word
#pragma unroll
        for (uint32_t step = 0; step < 2; ++step) {
          const uint32_t g = 2u * step + hi;
          uint32_t raw[kBlock][1];
#pragma unroll
          for (uint32_t k = 0; k < kBlock; ++k)
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(raw[k][0]) : "r"(box_chunk(box, g * kBlock + k, c) + wofs));
          float amax[2];
          column_amax<DTYPE, 2>(raw, amax);
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {
            const BlockScale s = block_scale<FMT>(amax[cc]);
            uint32_t cw[8];
            column_cast<FMT, ROUND, DTYPE, 2>(raw, cc, s, cw);
            pack6_words(cw, o[step][cc]);
            sb[cc] |= s.byte << (8 * g);
          }
        }
        const uint32_t kb = tr * 4u;
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
          // the run's 24 words: groups 0 and 2 in lane hi = 0 (o[0], o[1]), groups 1 and 3 in lane hi = 1.
          // sector 0 = g0[0..5] g1[0..1], sector 1 = g1[2..5] g2[0..3] (both written by hi = 0),
          // sector 2 = g2[4..5] g3[0..5] (written by hi = 1)
          uint32_t p1[6], p2[2];
#pragma unroll
          for (int i = 0; i < 6; ++i) p1[i] = __shfl_xor_sync(0xFFFFFFFFu, o[0][cc][i], 16);       // hi = 0 receives g1
#pragma unroll
          for (int i = 0; i < 2; ++i) p2[i] = __shfl_xor_sync(0xFFFFFFFFu, o[1][cc][4 + i], 16);   // hi = 1 receives g2[4..5]
          const uint32_t col = col0 + (warp >> 1) * 64u + w * 2u + cc;
          uint8_t* run0 = elems_col + (size_t)col * col_out_bytes + (size_t)kb * kBpb;
          const bool wide = (reinterpret_cast<uintptr_t>(run0) & 31u) == 0;
          if (hi == 0) {
            const uint32_t run[16] = {o[0][cc][0], o[0][cc][1], o[0][cc][2], o[0][cc][3], o[0][cc][4], o[0][cc][5],
                                      p1[0], p1[1], p1[2], p1[3], p1[4], p1[5],
                                      o[1][cc][0], o[1][cc][1], o[1][cc][2], o[1][cc][3]};
            store_run<16>(run0, run, wide);
          } else {
            const uint32_t run[8] = {p2[0], p2[1], o[1][cc][0], o[1][cc][1], o[1][cc][2], o[1][cc][3],
                                     o[1][cc][4], o[1][cc][5]};
            store_run<8>(run0 + 64, run, wide);
          }
          // the column's four scale bytes as one word (adjacent in either layout: kb % 4 == 0)
          const uint32_t word = sb[cc] | __shfl_xor_sync(0xFFFFFFFFu, sb[cc], 16);
          if (hi == 1) *reinterpret_cast<uint32_t*>(scales_col + scale_offset<LAYOUT>(col, kb, kb_col)) = word;
        }
      }
    }
    __syncwarp();
    if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar0 + 8 * (kStages + stage)) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------
// The same for FP32 input and 6-bit codes (configuration 4's tensors, whose register kernel needs
// six tile-times on a one-wave tensor where 4.6 would do).  An FP32 box row of 128 bytes is exactly
// one MX block, so a tile is four boxes side by side -- 128 x 128 elements, 64 KB, a row's four
// blocks = one 96-byte run --, three stages, one CTA per SM:
//   warps 0-3   rows: lane = one tile row, four blocks (eight 16-byte loads each)
//   warps 4-11  columns: warp w the w-th sixteenth... of the tile's 128 columns: lane = (column
//               lane % 16 of the warp's 16, row group 2 step + lane / 16), two steps; the two lanes of
//               a column then hold row groups {0, 2} and {1, 3} and pass eight words to each other
//               so that one writes sectors 0 and 1 of the column's 96-byte run and the other sector 2
//   warp 12     producer
// Rows convert 128 elements per lane and tile, columns 64: the twelve warps carry equal shares.
// ---------------------------------------------------------------------------------------------
constexpr uint32_t kTfBoxes = 4;
constexpr uint32_t kTfWarps = 12;
constexpr int kTileF32Threads = 32 * (kTfWarps + 1);
constexpr uint32_t kTfTileBytes = kTfBoxes * kBoxBytes;
constexpr uint32_t kTfCols = 32 * kTfBoxes;
constexpr uint32_t kTfStages = 3;
constexpr uint32_t kTfSmem = kTfStages * kTfTileBytes + 2 * kTfStages * 8 + kTfStages * 4 + 4 + 1024;

template <int FMT, int ROUND, int LAYOUT>
__global__ void __launch_bounds__(kTileF32Threads, 1)
quantize_tile_dual_f32_kernel(const __grid_constant__ CUtensorMap tmap_in, uint8_t* __restrict__ elems_row,
                              uint8_t* __restrict__ scales_row, uint8_t* __restrict__ elems_col,
                              uint8_t* __restrict__ scales_col, uint32_t R, uint32_t C, uint32_t tiles_c,
                              uint32_t num_tiles, uint32_t sched_slot) {
  static_assert(FmtTraits<FMT>::bits == 6, "6-bit codes");
  constexpr uint32_t kStages = kTfStages;
  constexpr uint32_t kBpb = 24;
  extern __shared__ uint8_t tile_smem_raw[];
  const uint32_t base = (smem_addr(tile_smem_raw) + 1023u) & ~1023u;
  const uint32_t bar0 = base + kStages * kTfTileBytes;      // landed[s] at 8 s, read[s] at 8 (kStages + s)
  const uint32_t tile_id0 = bar0 + 16 * kStages;
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    for (uint32_t s = 0; s < kStages; ++s) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar0 + 8 * s) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar0 + 8 * (kStages + s)), "r"(kTfWarps) : "memory");
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_in)) : "memory");
  }
  __syncthreads();
  pdl_prologue();
  const uint32_t kb_row = C / kBlock, kb_col = R / kBlock;
  const size_t row_out_bytes = (size_t)kb_row * kBpb, col_out_bytes = (size_t)kb_col * kBpb;
  if (warp == kTfWarps) {
    tile_producer<kStages, kTfBoxes>(&tmap_in, base, bar0, tile_id0, 32u, tiles_c, num_tiles, sched_slot, lane);
    return;
  }
#pragma unroll 1
  for (uint32_t it = 0;; ++it) {
    const uint32_t stage = it % kStages, parity = (it / kStages) & 1u;
    if (!tile_wait(bar0 + 8 * stage, parity)) {
      if (lane == 0) atomicCAS(&g_tile_status, 0u, 1u);
      return;
    }
    uint32_t t;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(t) : "r"(tile_id0 + 4 * stage) : "memory");
    if (t >= num_tiles) return;  // no tile left
    const uint32_t tr = t / tiles_c, tc = t - tr * tiles_c;
    const uint32_t tile_base = base + stage * kTfTileBytes;
    const uint32_t row0 = tr * kTileRows, col0 = tc * kTfCols;
    if (warp < 4u) {
      const uint32_t r = warp * 32u + lane;
      uint32_t run[24];
      uint32_t scale_word = 0;
#pragma unroll
      for (uint32_t q = 0; q < 4; ++q) {  // block q of the row = row r of box q
        const uint32_t box = tile_base + q * kBoxBytes;
        uint32_t u[32];
#pragma unroll
        for (uint32_t i = 0; i < 8; ++i) {
          uint32_t v0, v1, v2, v3;
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                       : "=r"(v0), "=r"(v1), "=r"(v2), "=r"(v3) : "r"(box_chunk(box, r, i)));
          u[4 * i] = v0; u[4 * i + 1] = v1; u[4 * i + 2] = v2; u[4 * i + 3] = v3;
        }
        float m[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) m[i] = absmax_nan(__uint_as_float(u[2 * i]), __uint_as_float(u[2 * i + 1]));
#pragma unroll
        for (int n = 8; n >= 1; n >>= 1)
#pragma unroll
          for (int i = 0; i < n; ++i) m[i] = absmax_nan(m[2 * i], m[2 * i + 1]);
        const BlockScale s = block_scale<FMT>(m[0]);
        scale_word |= s.byte << (8 * q);
        uint32_t cw[8], o[6];
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          float x[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) x[i] = __uint_as_float(u[8 * g + i]);
          cast8<FMT, ROUND>(x, s, cw[2 * g], cw[2 * g + 1]);
        }
        pack6_words(cw, o);
#pragma unroll
        for (int i = 0; i < 6; ++i) run[6 * q + i] = o[i];
      }
      const uint32_t row = row0 + r, kb0 = tc * 4u;
      uint8_t* dst = elems_row + (size_t)row * row_out_bytes + (size_t)kb0 * kBpb;
      store_run<24>(dst, run, (reinterpret_cast<uintptr_t>(dst) & 31u) == 0);
      // four adjacent bytes in either layout (kb0 % 4 == 0)
      *reinterpret_cast<uint32_t*>(scales_row + scale_offset<LAYOUT>(row, kb0, kb_row)) = scale_word;
    } else {
      const uint32_t cwarp = warp - 4u, hi = lane >> 4;
      const uint32_t w = 16u * (cwarp & 1u) + (lane & 15u);        // column (= word) inside the box
      const uint32_t box = tile_base + (cwarp >> 1) * kBoxBytes;
      const uint32_t c = w >> 2, wofs = (w & 3u) * 4u;
      uint32_t o[2][6];   // [step][word]: row group 2 step + hi
      uint32_t sb = 0;    // this lane's two scale bytes at their positions in the column's word
#pragma unroll
      for (uint32_t step = 0; step < 2; ++step) {
        const uint32_t g = 2u * step + hi;
        uint32_t raw[kBlock][1];
#pragma unroll
        for (uint32_t k = 0; k < kBlock; ++k)
          asm volatile("ld.shared.b32 %0, [%1];" : "=r"(raw[k][0]) : "r"(box_chunk(box, g * kBlock + k, c) + wofs));
        float amax[1];
        column_amax<MX_F32, 1>(raw, amax);
        const BlockScale s = block_scale<FMT>(amax[0]);
        uint32_t cw[8];
        column_cast<FMT, ROUND, MX_F32, 1>(raw, 0, s, cw);
        pack6_words(cw, o[step]);
        sb |= s.byte << (8 * g);
      }
      // the run's 24 words: groups 0 and 2 in lane hi = 0 (o[0], o[1]), groups 1 and 3 in lane hi = 1.
      // sector 0 = g0[0..5] g1[0..1], sector 1 = g1[2..5] g2[0..3] (both written by hi = 0),
      // sector 2 = g2[4..5] g3[0..5] (written by hi = 1)
      uint32_t p1[6], p2[2];
#pragma unroll
      for (int i = 0; i < 6; ++i) p1[i] = __shfl_xor_sync(0xFFFFFFFFu, o[0][i], 16);       // hi = 0 receives g1
#pragma unroll
      for (int i = 0; i < 2; ++i) p2[i] = __shfl_xor_sync(0xFFFFFFFFu, o[1][4 + i], 16);   // hi = 1 receives g2[4..5]
      const uint32_t col = col0 + (cwarp >> 1) * 32u + w, kb = tr * 4u;
      uint8_t* run0 = elems_col + (size_t)col * col_out_bytes + (size_t)kb * kBpb;
      const bool wide = (reinterpret_cast<uintptr_t>(run0) & 31u) == 0;
      if (hi == 0) {
        const uint32_t run[16] = {o[0][0], o[0][1], o[0][2], o[0][3], o[0][4], o[0][5], p1[0], p1[1],
                                  p1[2], p1[3], p1[4], p1[5], o[1][0], o[1][1], o[1][2], o[1][3]};
        store_run<16>(run0, run, wide);
      } else {
        const uint32_t run[8] = {p2[0], p2[1], o[1][0], o[1][1], o[1][2], o[1][3], o[1][4], o[1][5]};
        store_run<8>(run0 + 64, run, wide);
      }
      const uint32_t word = sb | __shfl_xor_sync(0xFFFFFFFFu, sb, 16);
      if (hi == 1) *reinterpret_cast<uint32_t*>(scales_col + scale_offset<LAYOUT>(col, kb, kb_col)) = word;
    }
    __syncwarp();
    if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar0 + 8 * (kStages + stage)) : "memory");
  }
}

template <int FMT, int ROUND, int LAYOUT>
cudaError_t launch_tile_f32_t(const DualArgs& a) {
  cudaError_t e;
  EncodeTiledFn fn = encode_fn(&e);
  if (!fn) return e;
  CUtensorMap map;
  const cuuint64_t dims[2] = {(cuuint64_t)a.C, (cuuint64_t)a.R};
  const cuuint64_t strides[1] = {(cuuint64_t)a.C * 4};
  const cuuint32_t box[2] = {32, kTileRows};
  if (!encode_cached(fn, &map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, a.in, dims, strides, box,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B))
    return cudaErrorInvalidValue;
  static bool attr_set[64] = {false};
  int dev = 0;
  e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  auto kernel = quantize_tile_dual_f32_kernel<FMT, ROUND, LAYOUT>;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTfSmem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  const uint32_t tiles_r = (uint32_t)(a.R / kTileRows), tiles_c = (uint32_t)(a.C / kTfCols);
  const uint32_t num_tiles = tiles_r * tiles_c;
  const uint32_t grid = num_tiles < (uint32_t)a.sm_count ? num_tiles : (uint32_t)a.sm_count;
  return launch_pdl(kernel, dim3(grid), dim3(kTileF32Threads), kTfSmem, a.stream, map, a.elems_row, a.scales_row,
                    a.elems_col, a.scales_col, (uint32_t)a.R, (uint32_t)a.C, tiles_c, num_tiles, next_sched_slot());
}

template <int FMT>
cudaError_t dispatch_tile_f32(const DualArgs& a) {
  if (a.rounding == MX_RHAZ)
    return a.layout == MX_SCALES_LINEAR ? launch_tile_f32_t<FMT, MX_RHAZ, MX_SCALES_LINEAR>(a)
                                        : launch_tile_f32_t<FMT, MX_RHAZ, MX_SCALES_SWIZZLED>(a);
  return a.layout == MX_SCALES_LINEAR ? launch_tile_f32_t<FMT, MX_RNE, MX_SCALES_LINEAR>(a)
                                      : launch_tile_f32_t<FMT, MX_RNE, MX_SCALES_SWIZZLED>(a);
}

template <int FMT, int ROUND, int LAYOUT, bool COLS_ONLY = false>
cudaError_t launch_tile_dual_t(const DualArgs& a) {
  cudaError_t e;
  EncodeTiledFn fn = encode_fn(&e);
  if (!fn) return e;
  CUtensorMap map;
  const cuuint64_t dims[2] = {(cuuint64_t)a.C, (cuuint64_t)a.R};
  const cuuint64_t strides[1] = {(cuuint64_t)a.C * 2};
  const cuuint32_t box[2] = {64, kTileRows};
  if (!encode_cached(fn, &map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.in, dims, strides, box,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B))
    return cudaErrorInvalidValue;
  constexpr uint32_t kSt = 3;
  constexpr uint32_t smem = kSt * kTdTileBytes + 2 * kSt * 8 + kSt * 4 + 4 + 1024;  // stages, barriers, tile numbers, alignment slack
  static bool attr_set[64] = {false};
  int dev = 0;
  e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  auto kernel = quantize_tile_dual_kernel<FMT, ROUND, LAYOUT, COLS_ONLY>;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  const uint32_t tiles_r = (uint32_t)(a.R / kTileRows), tiles_c = (uint32_t)(a.C / kTdCols);
  const uint32_t num_tiles = tiles_r * tiles_c;
  const uint32_t slots = (uint32_t)kTdCtasPerSm * (uint32_t)a.sm_count;
  const uint32_t grid = num_tiles < slots ? num_tiles : slots;
  const uint32_t sched_slot = next_sched_slot();
  return launch_pdl(kernel, dim3(grid), dim3(kTileDualThreads), smem, a.stream, map, a.elems_row, a.scales_row,
                    a.elems_col, a.scales_col, (uint32_t)a.R, (uint32_t)a.C, tiles_c, num_tiles, sched_slot);
}

template <int FMT>
cudaError_t dispatch_tile_dual(const DualArgs& a) {
  if (a.rounding == MX_RHAZ)
    return a.layout == MX_SCALES_LINEAR ? launch_tile_dual_t<FMT, MX_RHAZ, MX_SCALES_LINEAR>(a)
                                        : launch_tile_dual_t<FMT, MX_RHAZ, MX_SCALES_SWIZZLED>(a);
  return a.layout == MX_SCALES_LINEAR ? launch_tile_dual_t<FMT, MX_RNE, MX_SCALES_LINEAR>(a)
                                      : launch_tile_dual_t<FMT, MX_RNE, MX_SCALES_SWIZZLED>(a);
}

// The column-block tensor alone (6- and 4-bit codes): the same kernel without its row pass (6-bit: the row warps idle).
template <int FMT>
cudaError_t dispatch_tile_cols(const DualArgs& a) {
  if (a.rounding == MX_RHAZ)
    return a.layout == MX_SCALES_LINEAR ? launch_tile_dual_t<FMT, MX_RHAZ, MX_SCALES_LINEAR, true>(a)
                                        : launch_tile_dual_t<FMT, MX_RHAZ, MX_SCALES_SWIZZLED, true>(a);
  return a.layout == MX_SCALES_LINEAR ? launch_tile_dual_t<FMT, MX_RNE, MX_SCALES_LINEAR, true>(a)
                                      : launch_tile_dual_t<FMT, MX_RNE, MX_SCALES_SWIZZLED, true>(a);
}

}  // namespace

// BF16 input, R and C multiples of 128 (what mx_quantize_dual requires of BF16 tensors).
cudaError_t launch_quantize_tile(const DualArgs& a) {
  if (a.dtype != MX_BF16 || !a.elems_row || !a.elems_col) return cudaErrorInvalidValue;
  switch (a.fmt) {
    case MX_E4M3: return dispatch_tile_dual<MX_E4M3>(a);
    case MX_E5M2: return dispatch_tile_dual<MX_E5M2>(a);
    case MX_E3M2: return dispatch_tile_dual<MX_E3M2>(a);
    case MX_E2M3: return dispatch_tile_dual<MX_E2M3>(a);
    case MX_E2M1: return dispatch_tile_dual<MX_E2M1>(a);
    default: return dispatch_tile_dual<MX_INT8>(a);
  }
}

// FP32 input, 6-bit codes, R and C multiples of 128.
cudaError_t launch_quantize_tile_f32(const DualArgs& a) {
  if (a.dtype != MX_F32 || !a.elems_row || !a.elems_col) return cudaErrorInvalidValue;
  switch (a.fmt) {
    case MX_E3M2: return dispatch_tile_f32<MX_E3M2>(a);
    case MX_E2M3: return dispatch_tile_f32<MX_E2M3>(a);
    default: return cudaErrorInvalidValue;
  }
}

// The column-block tensor alone ([C x R], blocks along axis 0 of X[R x C]) for the sub-byte formats:
// mx_quantize along axis 0 of a 2-D BF16 tensor of whole tiles, where it beats the register kernels
// (measured on 4096 x 16384: 6-bit 30.2 against 35.1 us, 4-bit 28.2 against 29.2; 8192 x 8192: 4-bit
// 28.6 against 30.3; 8-bit codes are faster in the register kernel, 33.9 against 34.5).
cudaError_t launch_quantize_tile_cols(const DualArgs& a) {
  if (a.dtype != MX_BF16 || !a.elems_col || !a.scales_col) return cudaErrorInvalidValue;
  switch (a.fmt) {
    case MX_E3M2: return dispatch_tile_cols<MX_E3M2>(a);
    case MX_E2M3: return dispatch_tile_cols<MX_E2M3>(a);
    case MX_E2M1: return dispatch_tile_cols<MX_E2M1>(a);
    default: return cudaErrorInvalidValue;
  }
}

// Reads and clears the status word of the tile kernels (after synchronising the stream).
cudaError_t quantize_tile_status(cudaStream_t stream, unsigned int* status) {
  cudaError_t e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) return e;
  e = cudaMemcpyFromSymbol(status, g_tile_status, sizeof(unsigned int));
  if (e != cudaSuccess) return e;
  if (*status != 0) {
    const unsigned int zero = 0;
    e = cudaMemcpyToSymbol(g_tile_status, &zero, sizeof(unsigned int));
  }
  return e;
}

}  // namespace mx
