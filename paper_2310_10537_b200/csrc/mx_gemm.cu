// MX block-scaled GEMM on the 5th-generation tensor cores (Section 4.1 of arXiv
// 2310.10537: dot products of two MX operands, scalar-float output).
//
//   C[m,n] = sum_b X_A[m,b] X_B[n,b] sum_{i<32} P_A[m,32b+i] P_B[n,32b+i]
//
// One tcgen05.mma kind::mxf8f6f4 block_scale instruction multiplies a 128 x 32
// slab of A with a BN x 32 slab of B and applies one E8M0 scale per row of A and
// per row of B -- exactly one MX block (k = 32) deep -- accumulating in FP32 in
// tensor memory.
//
// Kernel structure (one CTA per SM, persistent over output tiles; three kernels: 128-row tiles,
// 256-row tiles on CTA pairs, and swapped operands for few rows of A):
//   warp 0    operand producer: packed A / B tiles by TMA (the sub-byte tensor-map types expand
//             FP6 / FP4 to one byte per element on the way in) -> shared-memory ring
//   warp 11   scale producer: the stage's 512-byte swizzled scale chunks -> shared memory, on a
//             barrier of their own
//   warp 10   scale copier: a stage's scale chunks shared -> tensor memory (tcgen05.cp), then
//             tcgen05.commit tells the MMA issuer
//   warp 1    MMA issuer: four MMAs per stage, tcgen05.commit releases the stage / publishes the
//             accumulator
//   warps 2-9 epilogue: tensor memory -> registers (the accumulator is released as soon as it is
//             in registers) -> FP32 or BF16 C through shared memory and TMA stores, or the
//             quantizing epilogue (C as an MX tensor), overlapping the next tile's MMAs
// The four issuing warps run their loops converged -- all lanes wait on the barriers -- and issue
// from the lane elect.sync picks (see elect_one).
// Every wait on an mbarrier is bounded; on expiry the kernel records a status
// word, raises a CTA-wide abort flag and every role falls through to the common
// exit, where tensor memory is released.
#include <cuda.h>  // CUtensorMap and enums only: the driver entry point is looked up at run time
#include <cuda_runtime.h>

#include <cstring>

#include "mx.h"
#include "mx_device.cuh"
#include "mx_launch.h"
#include "mx_tmap.h"

namespace mx {
namespace {

constexpr int BM = 128;         // rows of C per tile (= MMA M, one TMEM lane per row)
constexpr int BK = 128;         // K elements per pipeline stage: 4 MX blocks, 4 MMAs
constexpr int kMmaK = 32;       // K of one kind::mxf8f6f4 MMA = the MX block size
constexpr int kThreads = 384;   // 12 warps: producer, MMA issuer, 8 epilogue warps, scale copier, scale producer
constexpr int kTmemCols = 512;  // whole tensor memory of the SM (one CTA per SM)
constexpr long long kSpinLimit = 2000000000LL;  // default budget of a wait in cycles (~1 s)
constexpr uint32_t kNoDrop = 0xFFFFFFFFu;       // "failure drill off" value of the drop_fill argument

enum : unsigned int {
  ST_OK = 0,
  ST_PRODUCER_WAIT = 1,    // producer: stage never became empty
  ST_MMA_WAIT_FULL = 2,    // MMA issuer: stage never became full
  ST_MMA_WAIT_ACC = 3,     // MMA issuer: accumulator never drained
  ST_EPILOGUE_WAIT = 4,    // epilogue: accumulator never became full
  ST_SCALE_WAIT = 5,       // scale copier: stage never became full
  ST_SMEM_ALIGN = 6,       // shared memory window not aligned as the tight configuration needs
};

// First failure of any GEMM launch on this device since the last check (0 = none).
__device__ unsigned int g_gemm_status;

// Epilogue staging in shared memory: chunks of 32 rows x 16 columns of FP32 per warp.
constexpr uint32_t kEpiChunkCols = 16;
constexpr uint32_t kEpiChunkBytes = 32 * kEpiChunkCols * 4;
constexpr uint32_t kEpiBufs = 1;                                   // staging chunks per warp
constexpr uint32_t kEpiBytes = 8 * kEpiBufs * kEpiChunkBytes;     // eight epilogue warps

template <int BN>
struct Cfg {
  static_assert(BN == 128 || BN == 256, "tile width");
  static constexpr int kStages = BN == 256 ? 4 : 6;
  static constexpr int kAccStages = BN == 256 ? 1 : 2;
  static constexpr int kSfbChunks = BN / 128;  // 512-byte scale chunks (128 rows each) of B per stage
  static constexpr int kSfCols = 4 + 4 * kSfbChunks;       // TMEM columns of scales per stage
  static constexpr int kSfCol0 = kAccStages * BN;          // first scale column
  static constexpr uint32_t kABytes = BM * BK;             // one byte per element in shared memory
  static constexpr uint32_t kBBytes = BN * BK;
  static constexpr uint32_t kSfBytes = 512 * (1 + kSfbChunks);
  static constexpr uint32_t kOffA = 0;
  static constexpr uint32_t kOffB = kOffA + kStages * kABytes;
  static constexpr uint32_t kOffEpi = kOffB + kStages * kBBytes;   // 1024-byte aligned
  static constexpr uint32_t kOffSf = kOffEpi + kEpiBytes;
  static constexpr uint32_t kOffBar = kOffSf + kStages * kSfBytes;
  // barriers: full[S], empty[S], acc_full[A], acc_empty[A], scales_ready[S], scales_landed[S]; then
  // tmem slot + abort flag
  static constexpr uint32_t kNumBars = 4 * kStages + 2 * kAccStages;
  static constexpr uint32_t kSmemBytes = kOffBar + kNumBars * 8 + 16 + 1024;  // + alignment slack
  static_assert(kSfCol0 + kStages * kSfCols <= kTmemCols, "tensor memory budget");
  static_assert(kSmemBytes <= 232448, "shared memory budget");
};

// ---- PTX wrappers ------------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: false if the abort flag was raised or the cycle budget `limit` ran out.  Waits for
// one pipeline stage get the kernel's budget; waits for a whole tile (the accumulator hand-overs)
// get four times as much, so that when a stage never arrives it is the stage wait that reports it.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity,
                                          const volatile uint32_t* abort_flag, long long limit) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 31u) == 0) {
      if (*abort_flag != 0) return false;
      if (clock64() - t0 > limit) return false;
    }
  }
}
// Every copy of a stage (A tile, B tile, A scales, B scales) goes through a rank-3 tensor map.
// The warps that issue copies, tcgen05.cp, tcgen05.mma and tcgen05.commit run their loops converged
// and issue from the lane elect_one() picks: issued from inside a `lane == 0` branch each of
// these instructions cost its thread 58-69 clocks (their operands are uniform registers, which
// divergent code has to fill per instruction), and the MMA thread could not keep the tensor pipe fed.
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
// One lane of a converged warp (the pattern the compiler knows for single-thread instructions).
__device__ __forceinline__ bool elect_one() {
  uint32_t p;
  asm volatile(
      "{\n\t.reg .pred P;\n\t"
      "elect.sync _|P, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, P;\n\t}"
      : "=r"(p));
  return p != 0;
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
               ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_cp_scales(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc)
               : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc,
                                       uint32_t idesc, uint32_t sfa_tmem, uint32_t sfb_tmem,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale.scale_vec::1X [%0], %1, %2, %3, [%4], [%5], p;\n\t"
      "}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(sfa_tmem), "r"(sfb_tmem),
        "r"(accumulate) : "memory");
}
// Dense BF16 x BF16 -> FP32 (kind::f16, K = 16 per instruction): no scale operands.
__device__ __forceinline__ void tc_mma_dense(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc,
                                             uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t"
      "}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, "
      "%12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, "
      "%30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
        "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major operand tile with 128-byte rows
// in the 128-byte swizzle (the layout the TMA tensor map writes): 8-row groups
// are 1024 bytes apart.  Advancing K by one MMA (32 bytes) adds 2 to the
// start-address field.
__device__ __forceinline__ uint64_t operand_desc(uint32_t saddr) {
  const uint64_t lo = ((saddr & 0x3FFFFu) >> 4) | (1u << 16);            // address, LBO = 16 B
  const uint64_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);            // SBO, version 1, SWIZZLE_128B
  return lo | (hi << 32);
}
// Descriptor of one 512-byte scale chunk: 32 rows of 16 bytes, no swizzle,
// 8-row groups 128 bytes apart.
__device__ __forceinline__ uint64_t scale_desc(uint32_t saddr) {
  const uint64_t lo = ((saddr & 0x3FFFFu) >> 4);
  const uint64_t hi = (128u >> 4) | (1u << 14);
  return lo | (hi << 32);
}

// ---- epilogue: registers -> shared memory -> TMA store ---------------------------
// A thread holds one row of the accumulator, so direct global stores would touch 32
// different lines per warp instruction and crowd the L1 data path that also feeds the
// tensor core from shared memory.  Instead each warp stages 32 rows x 16 columns (2 KB,
// 64-byte rows in the 64-byte TMA swizzle, conflict-free 16-byte stores) and one lane
// hands the chunk to the TMA engine, which writes full lines and clips at the tensor edge.

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int x, int y, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(src) : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}

// r[j][i] = column 32 j + i of this thread's row (row0 + lane) starting at column col0 of C.
// A staging chunk is 32 rows x 64 bytes: 16 FP32 columns, or 32 BF16 columns (each FP32
// accumulator rounded to nearest even).
template <uint32_t kLoads>
__device__ __forceinline__ void store_rows(const uint32_t (&r)[kLoads][32], uint32_t stage_smem,
                                           const CUtensorMap* tmap_c, int col0, int row0,
                                           uint32_t valid_cols, uint32_t lane, uint32_t c_bf16) {
  if (lane == 0) bulk_wait_read<0>();  // chunks of the previous tile have left shared memory
  __syncwarp();
  if (c_bf16) {
#pragma unroll
    for (uint32_t q = 0; q < kLoads; ++q) {
      if (q * 32u < valid_cols) {
        const uint32_t buf = q % kEpiBufs;
        if (q >= kEpiBufs) {
          if (lane == 0) bulk_wait_read<(int)kEpiBufs - 1>();
          __syncwarp();
        }
        const uint32_t base = stage_smem + buf * kEpiChunkBytes + lane * 64;
#pragma unroll
        for (uint32_t c = 0; c < 4; ++c) {
          uint32_t w[4];
#pragma unroll
          for (uint32_t i = 0; i < 4; ++i)
            asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w[i])
                : "f"(__uint_as_float(r[q][8 * c + 2 * i + 1])), "f"(__uint_as_float(r[q][8 * c + 2 * i])));
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                       ::"r"(base + ((c ^ ((lane >> 1) & 3u)) << 4)), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3])
                       : "memory");
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) tma_store_2d(tmap_c, col0 + (int)(q * 32u), row0, stage_smem + buf * kEpiChunkBytes);
      }
    }
    return;
  }
#pragma unroll
  for (uint32_t q = 0; q < kLoads * 2; ++q) {
    if (q * kEpiChunkCols < valid_cols) {
      const uint32_t buf = q % kEpiBufs;
      if (q >= kEpiBufs) {
        if (lane == 0) bulk_wait_read<(int)kEpiBufs - 1>();
        __syncwarp();
      }
      const uint32_t base = stage_smem + buf * kEpiChunkBytes + lane * 64;
#pragma unroll
      for (uint32_t c = 0; c < 4; ++c) {
        const uint32_t* v = &r[q / 2][(q % 2) * 16 + 4 * c];
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                     ::"r"(base + ((c ^ ((lane >> 1) & 3u)) << 4)), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3])
                     : "memory");
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0)
        tma_store_2d(tmap_c, col0 + (int)(q * kEpiChunkCols), row0, stage_smem + buf * kEpiChunkBytes);
    }
  }
}

// What the epilogue does with a tile.
struct EpiArgs {
  uint32_t mode;     // 0: FP32 C through tmap_c, 1: BF16 C through tmap_c, 2: C as an MX tensor
  uint32_t fmt;      // mode 2: element format of the output
  uint32_t sticky;   // mode 2: 1 = ties away from zero (see cast_pair), 0 = ties to even
  uint8_t* elems;    // mode 2: packed codes [rows x N], blocks along N
  uint8_t* scales;   // mode 2: swizzled scale tensor, rows x N / 32
};

// Quantizes this thread's kLoads blocks of 32 consecutive columns of row `row` (Algorithm 1 on the
// FP32 accumulators, the same helpers as the quantize kernels) and writes their codes and scale
// bytes; col0 is a multiple of 32 * kLoads.
template <int FMT, uint32_t kLoads>
__device__ __forceinline__ void store_mx_fmt(const uint32_t (&r)[kLoads][32], const EpiArgs& epi,
                                             uint32_t row, uint32_t col0, uint32_t N) {
  constexpr uint32_t W = FmtTraits<FMT>::bits;  // 32-bit words of codes per block
  uint32_t w[kLoads * W];
  uint32_t sword = 0;
#pragma unroll
  for (uint32_t j = 0; j < kLoads; ++j) {
    float m[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) m[i] = absmax_nan(__uint_as_float(r[j][2 * i]), __uint_as_float(r[j][2 * i + 1]));
#pragma unroll
    for (int n = 8; n >= 1; n >>= 1)
#pragma unroll
      for (int i = 0; i < n; ++i) m[i] = absmax_nan(m[i], m[i + n]);
    const BlockScale bs = block_scale<FMT>(m[0]);
    sword |= bs.byte << (8 * j);
    uint32_t lo[4], hi[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      uint32_t p[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float a = mul_ftz(__uint_as_float(r[j][8 * g + 2 * i]), bs.m1);
        float b = mul_ftz(__uint_as_float(r[j][8 * g + 2 * i + 1]), bs.m1);
        if (FMT == MX_INT8) { a *= bs.m2; b *= bs.m2; }
        a = __uint_as_float(__float_as_uint(a) | epi.sticky);
        b = __uint_as_float(__float_as_uint(b) | epi.sticky);
        p[i] = cast_pair<FMT, MX_RNE>(a, b);
      }
      pack8<FMT>(p, lo[g], hi[g]);
      if (!bs.finite) { lo[g] = 0; hi[g] = 0; }
    }
    if (W == 8) {
#pragma unroll
      for (int g = 0; g < 4; ++g) { w[8 * j + 2 * g] = lo[g]; w[8 * j + 2 * g + 1] = hi[g]; }
    } else if (W == 4) {
#pragma unroll
      for (int g = 0; g < 4; ++g) w[4 * j + g] = lo[g];
    } else {  // 8 codes = 48 bits: two groups fill three words
      w[6 * j + 0] = lo[0];
      w[6 * j + 1] = __byte_perm(hi[0], lo[1], 0x5410);
      w[6 * j + 2] = __byte_perm(lo[1], hi[1], 0x5432);
      w[6 * j + 3] = lo[2];
      w[6 * j + 4] = __byte_perm(hi[2], lo[3], 0x5410);
      w[6 * j + 5] = __byte_perm(lo[3], hi[3], 0x5432);
    }
  }
  uint8_t* dst = epi.elems + ((size_t)row * N + col0) / 8 * W;
  store_run<(int)(kLoads * W)>(dst, w, (reinterpret_cast<uintptr_t>(dst) & 31u) == 0);
  // swizzled scale layout: the kLoads scale bytes of this row are adjacent inside one 512-byte chunk
  const uint32_t kb = col0 / 32;
  uint8_t* sp = epi.scales + ((size_t)(row / 128) * (N / 128) + kb / 4) * 512 + (row % 32) * 16 +
                ((row % 128) / 32) * 4 + kb % 4;
  if (kLoads == 4) *reinterpret_cast<uint32_t*>(sp) = sword;
  else *reinterpret_cast<uint16_t*>(sp) = (uint16_t)sword;
}

template <uint32_t kLoads>
__device__ __forceinline__ void store_mx_rows(const uint32_t (&r)[kLoads][32], const EpiArgs& epi,
                                              uint32_t row, uint32_t col0, uint32_t N) {
  static_assert(kLoads == 2 || kLoads == 4, "two or four blocks per thread");
  switch (epi.fmt) {
    case MX_E4M3: store_mx_fmt<MX_E4M3, kLoads>(r, epi, row, col0, N); break;
    case MX_E5M2: store_mx_fmt<MX_E5M2, kLoads>(r, epi, row, col0, N); break;
    case MX_E3M2: store_mx_fmt<MX_E3M2, kLoads>(r, epi, row, col0, N); break;
    case MX_E2M3: store_mx_fmt<MX_E2M3, kLoads>(r, epi, row, col0, N); break;
    case MX_E2M1: store_mx_fmt<MX_E2M1, kLoads>(r, epi, row, col0, N); break;
    default: store_mx_fmt<MX_INT8, kLoads>(r, epi, row, col0, N); break;
  }
}

struct TileCoord {
  uint32_t tm, tn, b;
};
// Output tiles are walked batch by batch and, inside a matrix, in bands of group_m tile rows so
// that the A band and the B tiles of a wave of CTAs stay in L2.
__device__ __forceinline__ TileCoord tile_coord(uint32_t t, uint32_t tiles_m, uint32_t tiles_n,
                                                uint32_t group_m) {
  TileCoord c;
  const uint32_t per_batch = tiles_m * tiles_n;
  c.b = t / per_batch;
  t -= c.b * per_batch;
  const uint32_t per_group = group_m * tiles_n;
  const uint32_t g = t / per_group, r = t - g * per_group;
  const uint32_t first_m = g * group_m;
  const uint32_t gm = min(group_m, tiles_m - first_m);
  c.tn = r / gm;
  c.tm = first_m + (r - c.tn * gm);
  return c;
}

__device__ __forceinline__ void raise_abort(volatile uint32_t* abort_flag, unsigned int code) {
  atomicCAS(&g_gemm_status, 0u, code);
  *abort_flag = 1u;
}

// Implicit-GEMM convolution (CONV): the A operand [N Ho Wo x kh kw C] is never materialized.  The
// activation x[N, H, W, C] was quantized once along C (8-bit codes), so block (m, kb) of A is block
// kb % (C / 32) of the input pixel that filter tap kb / (C / 32) of output pixel m reads -- or a zero
// block where the tap falls into the padding.  When C is a multiple of 128 a stage's 128 K elements
// lie in one filter tap and ONE copy through an im2col-mode tensor map brings the stage's 128 rows
// x 128 bytes (128 consecutive output pixels, their input pixels found by the copy engine, padding
// filled with zeros); otherwise four extra warps gather them with 16-byte cp.async copies straight
// into the 128-byte-swizzled operand layout.  In both cases those warps compose each row's four
// scale bytes into the stage's scale chunk.
struct ConvGeom {
  const uint8_t* x_codes;   // [N H W][C] codes, one byte each
  const uint8_t* x_scales;  // [N H W rows][C / 32]
  uint32_t H, W, Ho, Wo, kw, C, cb, kblocks, M, x_rows, x_layout;
  uint32_t tma;  // 1: the codes come through an im2col tensor map (C % 128 == 0), the gather warps only place scales
  int32_t stride_h, stride_w, pad_h, pad_w, dil_h, dil_w;
  FastDiv d_wo, d_howo, d_kw, d_cb;
};
constexpr int kConvThreads = kThreads + 128;  // + four gather warps
constexpr int kConvLag = 2;                   // stages a gather thread keeps in flight before it signals one

// 128 pixels x 128 channels of x[N, H, W, C] for one filter tap: (c, w, h, n) is the first channel
// and the input position that tap (0, 0) of the first output pixel reads, (ow, oh) the tap's offset.
__device__ __forceinline__ void tma_load_im2col(uint32_t dst, const CUtensorMap* map, int c, int w, int h, int n,
                                                uint32_t ow, uint32_t oh, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6], {%7, %8};"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c), "r"(w), "r"(h), "r"(n), "r"(bar),
        "h"((uint16_t)ow), "h"((uint16_t)oh) : "memory");
}

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}

// One scale word global -> shared without passing through a register (src_bytes 0: a zero word), and
// an arrival on a barrier of this CTA that happens when the thread's copies so far have landed
// (counted in the barrier's expected arrivals).  A thread that fetched the words through registers
// would have to order them with a release before signalling, and a release waits for every load the
// thread has in flight -- the ones it requested ahead included.
__device__ __forceinline__ void cp_async_4(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_arrive(uint32_t bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}

// DENSE: the operands are BF16 matrices (MX tensors dequantized beforehand, which is exact) and the
// MMA is the plain kind::f16 one: a stage holds 64 K-elements (the same 128-byte rows), no scales.
template <int BN, bool DENSE, bool CONV>
__device__ __forceinline__ void
gemm_kernel_body(const CUtensorMap& tmap_a, const CUtensorMap& tmap_b, const CUtensorMap& tmap_sa,
                 const CUtensorMap& tmap_sb, const CUtensorMap& tmap_c, uint32_t M, uint32_t N, uint32_t K,
                 uint32_t idesc_base, uint32_t group_m, uint32_t tx_bytes, EpiArgs epi, uint32_t batch,
                 long long spin_limit, uint32_t drop_fill, const ConvGeom& cg) {
  static_assert(!CONV || (!DENSE && BN == 128), "the gather warps fit the register budget of the 128-wide tile");
  using cfg = Cfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar0 = smem_base + cfg::kOffBar;
  auto full_bar = [&](uint32_t s) { return bar0 + 8 * s; };
  auto empty_bar = [&](uint32_t s) { return bar0 + 8 * (cfg::kStages + s); };
  auto acc_full_bar = [&](uint32_t a) { return bar0 + 8 * (2 * cfg::kStages + a); };
  auto acc_empty_bar = [&](uint32_t a) { return bar0 + 8 * (2 * cfg::kStages + cfg::kAccStages + a); };
  auto sf_ready_bar = [&](uint32_t s) { return bar0 + 8 * (2 * cfg::kStages + 2 * cfg::kAccStages + s); };
  auto sf_full_bar = [&](uint32_t s) { return bar0 + 8 * (3 * cfg::kStages + 2 * cfg::kAccStages + s); };
  volatile uint32_t* tmem_slot =
      reinterpret_cast<volatile uint32_t*>(smem_gen + cfg::kOffBar + cfg::kNumBars * 8);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tiles_m = (M + BM - 1) / BM, tiles_n = (N + BN - 1) / BN;
  const uint32_t num_tiles = batch * tiles_m * tiles_n;
  constexpr uint32_t BKe = DENSE ? 64 : BK;     // K elements per stage
  const uint32_t k_chunks = (K + BKe - 1) / BKe;  // a K tail is zero-filled by the copies

  if (threadIdx.x == 0) {
    for (uint32_t s = 0; s < cfg::kStages; ++s) {
      mbar_init(full_bar(s), (CONV && !cg.tma) ? 5 : 1);  // the producer's arrive + bytes (gathered codes: + one arrival per gather warp)
      mbar_init(empty_bar(s), 1);
      mbar_init(sf_ready_bar(s), 1);  // the copier's tcgen05.commit
      mbar_init(sf_full_bar(s), CONV ? (cg.tma ? 33 : 5) : 1);  // the scale producer's arrive + scale bytes (CONV: + the lanes of the warp that copies the A scale words, or the four gather warps)
    }
    for (uint32_t a = 0; a < cfg::kAccStages; ++a) {
      mbar_init(acc_full_bar(a), 1);
      mbar_init(acc_empty_bar(a), 8);  // one arrival per epilogue warp
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_a)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_b)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_c)) : "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))), "r"((uint32_t)kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // The kernel is launched with programmatic stream serialization: everything above then
  // overlapped the tail of the kernel before, and nothing below touches global memory before that
  // kernel has completed.  The kernel does not announce its own dependents early: CTAs of a
  // following kernel that wait on SMs this grid has already left slowed the rest of it down (a
  // chain of 4096^3 products and quantizes: +7 %).
  asm volatile("griddepcontrol.wait;" ::: "memory");

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    // The two operand copies of a stage; the scale chunks have a producer warp of their own (warp
    // 11).  The whole warp runs the loop converged and one elected lane issues (see elect_one).
    // Failure drill (drop_fill != kNoDrop): the fill with that running number is left out -- no copy
    // is issued and its barrier is not armed -- so that the MMA issuer's wait for it runs out.
    uint32_t stage = 0, phase = 0, fill = 0;
    bool ok = true;
    for (uint32_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
      const TileCoord tc = tile_coord(t, tiles_m, tiles_n, group_m);
      // (k, row, 0), rows counted through the whole batch.  Rows past the end of a B matrix on a
      // ragged last tile belong to the next matrix of the batch or are zero-filled by the copy;
      // their columns are not stored.
      const int cy_a = (int)((tc.b * tiles_m + tc.tm) * BM), cy_b = (int)(tc.b * N + tc.tn * BN);
      // CONV through the im2col map: where tap (0, 0) of the tile's first output pixel reads
      int cv_w = 0, cv_h = 0, cv_n = 0;
      if (CONV) {
        const uint32_t m0 = tc.tm * BM, n0 = fastdiv(m0, cg.d_howo), rem = m0 - n0 * (cg.Ho * cg.Wo);
        const uint32_t ho = fastdiv(rem, cg.d_wo), wo = rem - ho * cg.Wo;
        cv_n = (int)n0;
        cv_h = (int)ho * cg.stride_h - cg.pad_h;
        cv_w = (int)wo * cg.stride_w - cg.pad_w;
      }
      for (uint32_t kc = 0; kc < k_chunks; ++kc) {
        ok = __all_sync(0xffffffffu, mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, spin_limit));
        if (!ok) {
          raise_abort(abort_flag, ST_PRODUCER_WAIT);
          break;
        }
        if (fill++ != drop_fill && elect_one()) {
          const uint32_t fb = full_bar(stage);
          mbar_arrive_expect_tx(fb, tx_bytes);
          if (!CONV) {
            tma_load_3d(smem_base + cfg::kOffA + stage * cfg::kABytes, &tmap_a, (int)(kc * BKe), cy_a, 0, fb);
          } else if (cg.tma) {  // the stage's K chunk = 128 channels of one filter tap
            const uint32_t tap = fastdiv(kc * 4, cg.d_cb), cblk = kc * 4 - tap * cg.cb;
            const uint32_t ti = fastdiv(tap, cg.d_kw), tj = tap - ti * cg.kw;
            tma_load_im2col(smem_base + cfg::kOffA + stage * cfg::kABytes, &tmap_a, (int)(cblk * 32u), cv_w, cv_h, cv_n,
                            tj * (uint32_t)cg.dil_w, ti * (uint32_t)cg.dil_h, fb);
          }
          tma_load_3d(smem_base + cfg::kOffB + stage * cfg::kBBytes, &tmap_b, (int)(kc * BKe), cy_b, 0, fb);
        }
        __syncwarp();
        if (++stage == cfg::kStages) { stage = 0; phase ^= 1u; }
      }
    }
    if (!ok) {  // let copies that are still in flight land before the CTA goes away
      const long long t0 = clock64();
      while (clock64() - t0 < 2000000LL) {}
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer -------------------------------
    // the warp runs converged; one elected lane issues a stage's MMAs and the commit
    uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
    bool ok = true;
    for (uint32_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
      if (!__all_sync(0xffffffffu, mbar_wait(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag, 4 * spin_limit))) {
        raise_abort(abort_flag, ST_MMA_WAIT_ACC);
        break;
      }
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + acc * BN;
      // scales of row n of the tile sit in column (n0 % 128 + n) / 32 of the copied chunks
      const uint32_t sfb_col = 4 + ((tile_coord(t, tiles_m, tiles_n, group_m).tn * BN) % 128) / 32;
      for (uint32_t kc = 0; kc < k_chunks; ++kc) {
        // scales in tensor memory, then the operands
        ok = __all_sync(0xffffffffu, (DENSE || mbar_wait(sf_ready_bar(stage), phase, abort_flag, spin_limit)) &&
                                         mbar_wait(full_bar(stage), phase, abort_flag, spin_limit));
        if (!ok) {
          raise_abort(abort_flag, ST_MMA_WAIT_FULL);
          break;
        }
        tc_fence_after();
        const uint32_t sf_tmem = tmem_base + cfg::kSfCol0 + stage * cfg::kSfCols;
        const uint64_t adesc = operand_desc(smem_base + cfg::kOffA + stage * cfg::kABytes);
        const uint64_t bdesc = operand_desc(smem_base + cfg::kOffB + stage * cfg::kBBytes);
        if (elect_one()) {
#pragma unroll
          for (uint32_t k = 0; k < BK / kMmaK; ++k) {
            // byte k of each 32-bit scale column belongs to MX block k of this stage
            if (DENSE) {
              tc_mma_dense(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc_base, (kc | k) != 0 ? 1u : 0u);
            } else {
              const uint32_t idesc = idesc_base | (k << 4) | (k << 29);
              tc_mma(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, sf_tmem, sf_tmem + sfb_col,
                     (kc | k) != 0 ? 1u : 0u);
            }
          }
          tc_commit(empty_bar(stage));  // the stage is free once these MMAs have read it
        }
        __syncwarp();
        if (++stage == cfg::kStages) { stage = 0; phase ^= 1u; }
      }
      if (ok && elect_one()) tc_commit(acc_full_bar(acc));
      __syncwarp();
      if (++acc == cfg::kAccStages) { acc = 0; acc_phase ^= 1u; }
    }
  } else if (warp == 10) {
    // ------------------------------ scale copier ------------------------------
    if constexpr (!DENSE) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      for (uint32_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
        for (uint32_t kc = 0; kc < k_chunks; ++kc) {
          ok = __all_sync(0xffffffffu, mbar_wait(sf_full_bar(stage), phase, abort_flag, spin_limit));
          if (!ok) {
            raise_abort(abort_flag, ST_SCALE_WAIT);
            break;
          }
          if (CONV) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the A scale words were written by ordinary copies
          tc_fence_after();
          const uint32_t sf_smem = smem_base + cfg::kOffSf + stage * cfg::kSfBytes;
          const uint32_t sf_tmem = tmem_base + cfg::kSfCol0 + stage * cfg::kSfCols;
          if (elect_one()) {
            tc_cp_scales(sf_tmem, scale_desc(sf_smem));
#pragma unroll
            for (uint32_t j = 0; j < cfg::kSfbChunks; ++j)
              tc_cp_scales(sf_tmem + 4 + 4 * j, scale_desc(sf_smem + 512 + 512 * j));
            tc_commit(sf_ready_bar(stage));  // arrives when the copies above have completed
          }
          __syncwarp();
          if (++stage == cfg::kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 11) {
    // ----------------------------- scale producer -----------------------------
    // The A scales of the tile's 128 rows and the B scales of its BN columns -- (0, K chunk, 128-row
    // group), groups counted through the whole batch; both complete on the per-stage "scales
    // landed" barrier.  A stage's scale buffer and scale columns are free when the stage is.
    if constexpr (!DENSE) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      for (uint32_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
        const TileCoord tc = tile_coord(t, tiles_m, tiles_n, group_m);
        const int cz_a = (int)(tc.b * tiles_m + tc.tm), cz_b = (int)((tc.b * N + tc.tn * BN) / 128);
        for (uint32_t kc = 0; kc < k_chunks; ++kc) {
          ok = __all_sync(0xffffffffu, mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, spin_limit));
          if (!ok) {
            raise_abort(abort_flag, ST_PRODUCER_WAIT);
            break;
          }
          if (elect_one()) {
            const uint32_t fb = sf_full_bar(stage);
            mbar_arrive_expect_tx(fb, CONV ? cfg::kSfBytes - 512u : cfg::kSfBytes);
            const uint32_t dst = smem_base + cfg::kOffSf + stage * cfg::kSfBytes;
            if (!CONV) tma_load_3d(dst, &tmap_sa, 0, (int)kc, cz_a, fb);
            tma_load_3d(dst + 512u, &tmap_sb, 0, (int)kc, cz_b, fb);
          }
          __syncwarp();
          if (++stage == cfg::kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
      }
    }
  } else if (warp >= 12) {
    // ------------------- gather warps (CONV): thread r serves row r of the tile -------------------
    if constexpr (CONV) {
      if (cg.tma) {
        // The codes come through the im2col map; warp 12 alone copies the A scale words (lane l: rows
        // l, l + 32, l + 64, l + 96), asynchronously, each lane's arrival following its copies.
        if (warp == 12) {
          uint32_t stage = 0, phase = 0;
          bool ok = true;
          for (uint32_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
            const TileCoord tc = tile_coord(t, tiles_m, tiles_n, group_m);
            int32_t cvh[4], cvw[4];
            uint32_t cvp[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const uint32_t m = tc.tm * BM + lane + 32 * j;
              const uint32_t n0 = fastdiv(m, cg.d_howo), rem = m - n0 * (cg.Ho * cg.Wo);
              const uint32_t ho = fastdiv(rem, cg.d_wo), wo = rem - ho * cg.Wo;
              cvh[j] = (int32_t)ho * cg.stride_h - cg.pad_h;
              cvw[j] = (int32_t)wo * cg.stride_w - cg.pad_w;
              cvp[j] = m < cg.M ? n0 * cg.H * cg.W : 0xFFFFFFFFu;
            }
            for (uint32_t kc = 0; kc < k_chunks; ++kc) {
              ok = __all_sync(0xffffffffu, mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, spin_limit));
              if (!ok) {
                raise_abort(abort_flag, ST_PRODUCER_WAIT);
                break;
              }
              const uint32_t dst = smem_base + cfg::kOffSf + stage * cfg::kSfBytes;
              const uint32_t tap = fastdiv(kc * 4, cg.d_cb), cblk = kc * 4 - tap * cg.cb;
              const uint32_t ti = fastdiv(tap, cg.d_kw), tj = tap - ti * cg.kw;
              const int32_t dh = (int32_t)ti * cg.dil_h, dw = (int32_t)tj * cg.dil_w;
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int32_t hi = cvh[j] + dh, wi = cvw[j] + dw;
                const bool live = cvp[j] != 0xFFFFFFFFu && hi >= 0 && hi < (int32_t)cg.H && wi >= 0 && wi < (int32_t)cg.W;
                const uint32_t px = live ? cvp[j] + (uint32_t)hi * cg.W + (uint32_t)wi : 0u;
                const size_t so = cg.x_layout == MX_SCALES_LINEAR ? (size_t)px * cg.cb + cblk
                                                                  : scale_offset<MX_SCALES_SWIZZLED>(px, cblk, cg.cb);
                cp_async_4(dst + lane * 16u + (uint32_t)j * 4u, cg.x_scales + (live ? so : 0), live ? 4u : 0u);
              }
              cp_async_arrive(sf_full_bar(stage));
              if (++stage == cfg::kStages) { stage = 0; phase ^= 1u; }
            }
          }
          asm volatile("cp.async.wait_all;" ::: "memory");
        }
      } else {
      // Codes: thread (p, q) copies 16-byte chunk p of rows q, q + 16, ..., q + 112, so that one
      // warp instruction moves four whole 128-byte rows (four input pixels' channel runs: full
      // lines from L2, conflict-free rows in shared memory).  Scales: thread r composes the word
      // of row r.
      const uint32_t gt = threadIdx.x - (uint32_t)kThreads;
      const uint32_t p = gt & 7u, q = gt >> 3;
      uint32_t stage = 0, phase = 0, issued = 0, signalled = 0;
      bool ok = true;
      // a stage's codes are signalled kConvLag stages after they were requested: the copies of the
      // stages in between are then in flight, and the thread itself makes them visible to the
      // tensor core's proxy before its warp arrives (one arrival per warp: 128 arrivals on one
      // barrier word would serialise)
      auto signal_oldest = [&]() {
        const uint32_t st = signalled % cfg::kStages;
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(full_bar(st));
        ++signalled;
      };
      // C a multiple of 128: the four blocks of a stage belong to one filter tap, their scale
      // bytes are one aligned word
      const bool one_tap = (cg.cb & 3u) == 0;
      struct RowGeom {
        int32_t h0, w0;   // input coordinates of tap (0, 0)
        uint32_t pix0;    // first pixel of the row's image; 0xFFFFFFFF: row past M
      };
      auto row_geom = [&](uint32_t m) -> RowGeom {
        RowGeom g;
        const uint32_t n = fastdiv(m, cg.d_howo), rem = m - n * (cg.Ho * cg.Wo);
        const uint32_t ho = fastdiv(rem, cg.d_wo), wo = rem - ho * cg.Wo;
        g.h0 = (int32_t)ho * cg.stride_h - cg.pad_h;
        g.w0 = (int32_t)wo * cg.stride_w - cg.pad_w;
        g.pix0 = m < cg.M ? n * cg.H * cg.W : 0xFFFFFFFFu;
        return g;
      };
      // MX block kb of the reduction axis (kh, kw, C): filter tap offsets and channel block
      struct Tap {
        int32_t dh, dw;
        uint32_t cblk;
        bool ok;
      };
      auto tap_of = [&](uint32_t kb) -> Tap {
        Tap tp;
        const uint32_t tap = fastdiv(kb, cg.d_cb);
        tp.cblk = kb - tap * cg.cb;
        const uint32_t ti = fastdiv(tap, cg.d_kw), tj = tap - ti * cg.kw;
        tp.dh = (int32_t)ti * cg.dil_h;
        tp.dw = (int32_t)tj * cg.dil_w;
        tp.ok = kb < cg.kblocks;
        return tp;
      };
      // input pixel a row reads through a tap; false where the tap falls into the padding
      auto source = [&](const RowGeom& g, const Tap& tp, uint32_t& px) -> bool {
        const int32_t hi = g.h0 + tp.dh, wi = g.w0 + tp.dw;
        const bool live = tp.ok && g.pix0 != 0xFFFFFFFFu && hi >= 0 && hi < (int32_t)cg.H && wi >= 0 && wi < (int32_t)cg.W;
        px = live ? g.pix0 + (uint32_t)hi * cg.W + (uint32_t)wi : 0u;
        return live;
      };
      auto scale_at = [&](uint32_t px, uint32_t cblk) -> const uint8_t* {
        return cg.x_scales + (cg.x_layout == MX_SCALES_LINEAR ? (size_t)px * cg.cb + cblk
                                                              : scale_offset<MX_SCALES_SWIZZLED>(px, cblk, cg.cb));
      };
      for (uint32_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
        const TileCoord tc = tile_coord(t, tiles_m, tiles_n, group_m);
        RowGeom rows[8];
#pragma unroll
        for (uint32_t i = 0; i < 8; ++i) rows[i] = row_geom(tc.tm * BM + q + 16 * i);
        const RowGeom mine = row_geom(tc.tm * BM + gt);  // the row whose scale word this thread writes
        // the four scale bytes of K chunk kc of that row (requested one chunk ahead of their use)
        auto scale_word = [&](uint32_t kc) -> uint32_t {
          uint32_t px, word = 0;
          if (one_tap) {
            const Tap tp = tap_of(kc * 4);
            if (source(mine, tp, px)) word = __ldg(reinterpret_cast<const uint32_t*>(scale_at(px, tp.cblk)));
          } else {
#pragma unroll
            for (uint32_t b = 0; b < 4; ++b) {
              const Tap tp = tap_of(kc * 4 + b);
              if (source(mine, tp, px)) word |= (uint32_t)__ldg(scale_at(px, tp.cblk)) << (8 * b);
            }
          }
          return word;
        };
        // requested kScaleAhead K chunks before their use: a load takes longer than a stage
        constexpr uint32_t kScaleAhead = 4;
        uint32_t sword_queue[kScaleAhead] = {};
#pragma unroll
        for (uint32_t d = 0; d < kScaleAhead; ++d)
          if (d < k_chunks) sword_queue[d] = scale_word(d);
        // (unrolled by the queue depth: every queue slot is a fixed register, see the pair kernel)
        for (uint32_t kc0 = 0; kc0 < k_chunks && ok; kc0 += kScaleAhead) {
#pragma unroll
        for (uint32_t d = 0; d < kScaleAhead; ++d) {
          const uint32_t kc = kc0 + d;
          if (kc >= k_chunks || !ok) break;
          ok = __all_sync(0xffffffffu, mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, spin_limit));
          if (!ok) {
            raise_abort(abort_flag, ST_PRODUCER_WAIT);
            break;
          }
          if (!cg.tma) {
            const uint32_t a_base = smem_base + cfg::kOffA + stage * cfg::kABytes;
            const Tap tp = tap_of(kc * 4 + (p >> 1));  // the block chunk p lies in
            const uint32_t in_block = tp.cblk * 32u + (p & 1u) * 16u;
            // zero blocks (padding taps, rows past M, K tail) are written by copies of zero source bytes
#pragma unroll
            for (uint32_t i = 0; i < 8; ++i) {
              const uint32_t row = q + 16 * i;
              uint32_t px;
              const bool live = source(rows[i], tp, px);
              cp_async_16(a_base + row * 128u + ((p ^ (row & 7u)) << 4),
                          live ? cg.x_codes + (size_t)px * cg.C + in_block : cg.x_codes, live ? 16u : 0u);
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
          }
          const uint32_t sword = sword_queue[d];
          if (kc + kScaleAhead < k_chunks) sword_queue[d] = scale_word(kc + kScaleAhead);
          // row gt's four scale bytes, where the swizzled chunk keeps them
          asm volatile("st.shared.b32 [%0], %1;" ::"r"(smem_base + cfg::kOffSf + stage * cfg::kSfBytes +
                                                      (gt & 31u) * 16u + (gt >> 5) * 4u), "r"(sword) : "memory");
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive(sf_full_bar(stage));
          if (!cg.tma) {
            ++issued;
            if (issued - signalled > (uint32_t)kConvLag) {
              asm volatile("cp.async.wait_group %0;" ::"n"(kConvLag) : "memory");
              signal_oldest();
            }
          }
          if (++stage == cfg::kStages) { stage = 0; phase ^= 1u; }
        }
        }
      }
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      if (ok) {
        while (signalled < issued) signal_oldest();
      }
      }
    }
  } else {
    // -------------------------------- epilogue --------------------------------
    // Two warps per TMEM lane quarter, each taking half of the tile's columns into registers;
    // the accumulator is handed back before the global stores are issued.
    const uint32_t quarter = warp & 3u;           // TMEM lanes this warp may read: 32*quarter .. +31
    const uint32_t half = (warp - 2u) >> 2;       // 0: columns [0, BN/2), 1: [BN/2, BN)
    constexpr uint32_t kHalf = BN / 2, kLoads = kHalf / 32;
    uint32_t acc = 0, acc_phase = 0;
    for (uint32_t t = blockIdx.x; t < num_tiles; t += gridDim.x) {
      const TileCoord tc = tile_coord(t, tiles_m, tiles_n, group_m);
      if (!mbar_wait(acc_full_bar(acc), acc_phase, abort_flag, 4 * spin_limit)) {
        if (lane == 0) raise_abort(abort_flag, ST_EPILOGUE_WAIT);
        break;
      }
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((quarter * 32u) << 16) + acc * BN + half * kHalf;
      const uint32_t col0 = tc.tn * BN + half * kHalf;
      const uint32_t row0 = (tc.b * tiles_m + tc.tm) * BM + quarter * 32;
      // columns of this half that exist; nothing is stored for rows past the end of a last,
      // partial row tile (only a single matrix can have one: its rows end at M)
      const uint32_t valid_cols = (col0 < N && row0 < batch * M) ? min(kHalf, N - col0) : 0u;
      uint32_t r[kLoads][32];
#pragma unroll
      for (uint32_t j = 0; j < kLoads; ++j) tc_ld32(taddr + 32 * j, r[j]);
      tc_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty_bar(acc));  // the MMA issuer may overwrite the accumulator
      if (epi.mode == 2) {
        if (valid_cols) store_mx_rows<kLoads>(r, epi, row0 + lane, col0, N);
      } else {
        store_rows<kLoads>(r, smem_base + cfg::kOffEpi + (warp - 2u) * kEpiBufs * kEpiChunkBytes, &tmap_c,
                           (int)col0, (int)row0, valid_cols, lane, epi.mode);
      }
      if (++acc == cfg::kAccStages) { acc = 0; acc_phase ^= 1u; }
    }
    if (lane == 0) bulk_wait_read<0>();  // the stores have left shared memory; the kernel's end orders the writes
  }

  // common exit: every role arrives here, also after an abort
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"((uint32_t)kTmemCols) : "memory");
  }
}

template <int BN, bool DENSE>
__global__ void __launch_bounds__(kThreads, 1)
mx_gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
               const __grid_constant__ CUtensorMap tmap_sa, const __grid_constant__ CUtensorMap tmap_sb,
               const __grid_constant__ CUtensorMap tmap_c,
               uint32_t M, uint32_t N, uint32_t K, uint32_t idesc_base,
               uint32_t group_m, uint32_t tx_bytes, EpiArgs epi, uint32_t batch,
               long long spin_limit, uint32_t drop_fill) {
  const ConvGeom none = {};
  gemm_kernel_body<BN, DENSE, false>(tmap_a, tmap_b, tmap_sa, tmap_sb, tmap_c, M, N, K, idesc_base, group_m, tx_bytes,
                                     epi, batch, spin_limit, drop_fill, none);
}

// Implicit-GEMM convolution: the same kernel with four gather warps in place of the A copies
// (tmap_b / tmap_sb: the filter [Cout x kh kw C] and its scales; M = N Ho Wo, N = Cout, K = kh kw C).
__global__ void __launch_bounds__(kConvThreads, 1)
mx_conv_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_b,
               const __grid_constant__ CUtensorMap tmap_sb, const __grid_constant__ CUtensorMap tmap_c, uint32_t M,
               uint32_t N, uint32_t K, uint32_t idesc_base, uint32_t group_m, uint32_t tx_bytes, EpiArgs epi,
               long long spin_limit, const __grid_constant__ ConvGeom cg) {
  // tmap_x: the im2col-mode map over x's codes (cg.tma), else any valid map (unused)
  gemm_kernel_body<128, false, true>(tmap_x, tmap_b, tmap_sb, tmap_sb, tmap_c, M, N, K, idesc_base, group_m, tx_bytes,
                                     epi, 1u, spin_limit, kNoDrop, cg);
}


// ============================================================================
// Few rows of A (M <= 128; a decode step: a handful of activation rows against a weight matrix).
// The product is bound by reading B once from HBM, and what a CTA can have in flight is bounded by
// its shared memory, so the operands change places: the tile's 128 rows of B take the M side of
// the MMA (one TMEM lane per row of B) and the MP = M rounded up to 16 rows of A its N side.  A
// K chunk is then 16 KB of B + MP x 128 bytes of A instead of 16 KB + 16 KB; a stage holds two
// chunks and the ring up to six stages.  The accumulator is C transposed -- lane = column n of C, column = row m --
// which the epilogue writes with plain stores: for every m the 32 lanes of a warp store 32
// consecutive columns.
// Warps: 0 operand producer, 1 MMA issuer, 2..5 epilogue (one per TMEM lane quarter), 10 scale
// copier, 11 scale producer; two accumulator stages.
// ============================================================================
constexpr uint32_t kSkinnyMaxStages = 12;
constexpr uint32_t kSkinnyBars = 4 * kSkinnyMaxStages + 4;
// Tensor memory of the few-rows kernel: two accumulators of MP columns, `acc_stride` columns apart,
// and 8 scale columns per K chunk of every stage behind them.  One CTA per SM takes all 512 columns
// (accumulators at 0 and 128, scales from 256); where two CTAs share an SM (MP <= 96) each takes 256
// (accumulators at 0 and 96, scales from 192).
struct SkinnyTmem {
  uint32_t cols, acc_stride, sf_col0;
};

__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, "
      "%12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
mx_gemm_skinny_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x,
                      const __grid_constant__ CUtensorMap tmap_sw, const __grid_constant__ CUtensorMap tmap_sx,
                      void* __restrict__ C, uint32_t M, uint32_t N, uint32_t K, uint32_t MP,
                      uint32_t idesc_base, uint32_t tx_bytes, uint32_t stages, uint32_t kch, uint32_t c_bf16,
                      long long spin_limit, uint32_t drop_fill, SkinnyTmem tm) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  // a stage holds kch K chunks of 128 elements (two where the weights are sub-byte codes: their
  // chunk is half the HBM bytes for the same per-stage hand-shakes)
  const uint32_t x_bytes = MP * 128u;                 // per K chunk
  const uint32_t w_stage = kch * 16384u, x_stage = kch * x_bytes, sf_stage = kch * 1024u;
  const uint32_t off_x = stages * w_stage;
  const uint32_t off_sf = off_x + stages * x_stage;
  const uint32_t off_bar = off_sf + stages * sf_stage;
  const uint32_t bar0 = smem_base + off_bar;
  auto full_bar = [&](uint32_t s) { return bar0 + 8 * s; };
  auto empty_bar = [&](uint32_t s) { return bar0 + 8 * (kSkinnyMaxStages + s); };
  auto sf_ready_bar = [&](uint32_t s) { return bar0 + 8 * (2 * kSkinnyMaxStages + s); };
  auto sf_full_bar = [&](uint32_t s) { return bar0 + 8 * (3 * kSkinnyMaxStages + s); };
  auto acc_full_bar = [&](uint32_t a) { return bar0 + 8 * (4 * kSkinnyMaxStages + a); };
  auto acc_empty_bar = [&](uint32_t a) { return bar0 + 8 * (4 * kSkinnyMaxStages + 2 + a); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + off_bar + kSkinnyBars * 8);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tiles_n = (N + 127u) / 128u;
  const uint32_t k_chunks = ((K + BK - 1) / BK + kch - 1) / kch;  // stages per tile; a K tail is zero-filled by the copies

  if (threadIdx.x == 0) {
    for (uint32_t s = 0; s < stages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
      mbar_init(sf_ready_bar(s), 1);
      mbar_init(sf_full_bar(s), 1);
    }
    for (uint32_t a = 0; a < 2; ++a) {
      mbar_init(acc_full_bar(a), 1);
      mbar_init(acc_empty_bar(a), 4);  // one arrival per epilogue warp
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_w)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_x)) : "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))), "r"(tm.cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // The kernel is launched with programmatic stream serialization: everything above then
  // overlapped the tail of the kernel before, and nothing below touches global memory before that
  // kernel has completed.  The kernel does not announce its own dependents early: CTAs of a
  // following kernel that wait on SMs this grid has already left slowed the rest of it down (a
  // chain of 4096^3 products and quantizes: +7 %).
  asm volatile("griddepcontrol.wait;" ::: "memory");

  if (warp == 0 || warp == 11) {
    // ---------------- producers: warp 0 the operand boxes, warp 11 the scale chunks ----------------
    // The tile's 128 rows of B and all MP rows of A (or their scale chunks).  Rows past N or M are
    // zero-filled by the copy: zero codes, value +0.  The warp runs converged, one elected lane issues.
    const bool scales = warp == 11;
    uint32_t stage = 0, phase = 0, fill = 0;  // drop_fill: see the operand producer of mx_gemm_kernel
    bool ok = true;
    for (uint32_t t = blockIdx.x; t < tiles_n && ok; t += gridDim.x) {
      for (uint32_t kc = 0; kc < k_chunks; ++kc) {
        ok = __all_sync(0xffffffffu, mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, spin_limit));
        if (!ok) {
          raise_abort(abort_flag, ST_PRODUCER_WAIT);
          break;
        }
        if ((scales || fill++ != drop_fill) && elect_one()) {
          if (scales) {  // (0, K chunk, 128-row group); a chunk past K is zero-filled like a tail
            const uint32_t fb = sf_full_bar(stage);
            mbar_arrive_expect_tx(fb, sf_stage);
            for (uint32_t c = 0; c < kch; ++c) {
              const uint32_t dst = smem_base + off_sf + stage * sf_stage + c * 1024u;
              tma_load_3d(dst, &tmap_sw, 0, (int)(kc * kch + c), (int)t, fb);
              tma_load_3d(dst + 512u, &tmap_sx, 0, (int)(kc * kch + c), 0, fb);
            }
          } else {  // (k, row, 0)
            const uint32_t fb = full_bar(stage);
            mbar_arrive_expect_tx(fb, kch * tx_bytes);
            for (uint32_t c = 0; c < kch; ++c) {
              const int kx = (int)((kc * kch + c) * BK);
              tma_load_3d(smem_base + stage * w_stage + c * 16384u, &tmap_w, kx, (int)(t * 128u), 0, fb);
              tma_load_3d(smem_base + off_x + stage * x_stage + c * x_bytes, &tmap_x, kx, 0, 0, fb);
            }
          }
        }
        __syncwarp();
        if (++stage == stages) { stage = 0; phase ^= 1u; }
      }
    }
    if (!ok) {  // let copies that are still in flight land before the CTA goes away
      const long long t0 = clock64();
      while (clock64() - t0 < 2000000LL) {}
    }
  } else if (warp == 10) {
    // ------------------------------ scale copier ------------------------------
    uint32_t stage = 0, phase = 0;
    bool ok = true;
    for (uint32_t t = blockIdx.x; t < tiles_n && ok; t += gridDim.x) {
      for (uint32_t kc = 0; kc < k_chunks; ++kc) {
        ok = __all_sync(0xffffffffu, mbar_wait(sf_full_bar(stage), phase, abort_flag, spin_limit));
        if (!ok) {
          raise_abort(abort_flag, ST_SCALE_WAIT);
          break;
        }
        tc_fence_after();
        const uint32_t sf_smem = smem_base + off_sf + stage * sf_stage;
        const uint32_t sf_tmem = tmem_base + tm.sf_col0 + stage * 8u * kch;
        if (elect_one()) {
          for (uint32_t c = 0; c < kch; ++c) {
            tc_cp_scales(sf_tmem + 8 * c, scale_desc(sf_smem + 1024 * c));            // rows of B: the MMA's A-side scales
            tc_cp_scales(sf_tmem + 8 * c + 4, scale_desc(sf_smem + 1024 * c + 512));  // rows of A: its B-side scales
          }
          tc_commit(sf_ready_bar(stage));
        }
        __syncwarp();
        if (++stage == stages) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer -------------------------------
    uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
    bool ok = true;
    for (uint32_t t = blockIdx.x; t < tiles_n && ok; t += gridDim.x) {
      if (!__all_sync(0xffffffffu, mbar_wait(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag, 4 * spin_limit))) {
        raise_abort(abort_flag, ST_MMA_WAIT_ACC);
        break;
      }
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + acc * tm.acc_stride;
      for (uint32_t kc = 0; kc < k_chunks; ++kc) {
        ok = __all_sync(0xffffffffu, mbar_wait(sf_ready_bar(stage), phase, abort_flag, spin_limit) &&
                                         mbar_wait(full_bar(stage), phase, abort_flag, spin_limit));
        if (!ok) {
          raise_abort(abort_flag, ST_MMA_WAIT_FULL);
          break;
        }
        tc_fence_after();
        if (elect_one()) {
          for (uint32_t c = 0; c < kch; ++c) {
            const uint32_t sf_tmem = tmem_base + tm.sf_col0 + stage * 8u * kch + 8 * c;
            const uint64_t wdesc = operand_desc(smem_base + stage * w_stage + c * 16384u);
            const uint64_t xdesc = operand_desc(smem_base + off_x + stage * x_stage + c * x_bytes);
#pragma unroll
            for (uint32_t k = 0; k < BK / kMmaK; ++k) {
              // byte k of each 32-bit scale column belongs to MX block k of this chunk
              const uint32_t idesc = idesc_base | (k << 4) | (k << 29);
              tc_mma(d_tmem, wdesc + 2 * k, xdesc + 2 * k, idesc, sf_tmem, sf_tmem + 4, (kc | c | k) != 0 ? 1u : 0u);
            }
          }
          tc_commit(empty_bar(stage));
        }
        __syncwarp();
        if (++stage == stages) { stage = 0; phase ^= 1u; }
      }
      if (ok && elect_one()) tc_commit(acc_full_bar(acc));
      __syncwarp();
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  } else if (warp >= 2 && warp < 6) {
    // -------------------------------- epilogue --------------------------------
    const uint32_t quarter = warp & 3u;  // TMEM lanes this warp may read: 32 * quarter .. + 31
    uint32_t acc = 0, acc_phase = 0;
    for (uint32_t t = blockIdx.x; t < tiles_n; t += gridDim.x) {
      if (!mbar_wait(acc_full_bar(acc), acc_phase, abort_flag, 4 * spin_limit)) {
        if (lane == 0) raise_abort(abort_flag, ST_EPILOGUE_WAIT);
        break;
      }
      tc_fence_after();
      const uint32_t n = t * 128u + quarter * 32u + lane;  // this thread's column of C
      const uint32_t taddr = tmem_base + ((quarter * 32u) << 16) + acc * tm.acc_stride;
      for (uint32_t c = 0; c < MP; c += 16) {
        uint32_t r[16];
        tc_ld16(taddr + c, r);
        tc_wait_ld();
        if (c + 16 >= MP) {  // the accumulator is in registers: hand it back before the stores
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(acc_empty_bar(acc));
        }
        if (n < N) {
#pragma unroll
          for (uint32_t j = 0; j < 16; ++j) {
            const uint32_t m = c + j;
            if (m < M) {
              const size_t idx = (size_t)m * N + n;
              if (c_bf16) {
                uint16_t h;
                asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(h) : "f"(__uint_as_float(r[j])));
                reinterpret_cast<uint16_t*>(C)[idx] = h;
              } else
                reinterpret_cast<float*>(C)[idx] = __uint_as_float(r[j]);
            }
          }
        }
      }
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

  // common exit: every role falls through to here, also after a wait that gave up
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"(tm.cols) : "memory");
  }
}

// ============================================================================
// Two-CTA variant: a cluster of two CTAs (two SMs) computes one 256 x 256 tile
// with tcgen05.mma.cta_group::2.  CTA r of the pair stages rows 128r.. of the A
// tile and rows 128r.. of the B tile, so each SM moves half of B through its
// shared memory per flop compared with the one-CTA kernel.  The even CTA (the
// leader) issues every MMA; its accumulator rows 0..127 live in its own tensor
// memory, rows 128..255 in the peer's.
//   - both producers copy with the mbarrier of the LEADER as completion target
//     (cp.async.bulk.tensor ... .cta_group::2), the leader alone arms it with the
//     byte count of both CTAs;
//   - tcgen05.commit with a two-CTA mask releases a stage / publishes the
//     accumulator in both CTAs;
//   - the epilogue warps of both CTAs arrive on the leader's accumulator-empty
//     barrier.
// No load is multicast: each CTA fetches what it needs itself (the B scales are
// fetched by both).
// ============================================================================

// F4 = both operands FP4 E2M1: kind::mxf4 takes them densely packed (two codes per byte, K = 64 per
// MMA, two MX blocks and therefore two scales per row and instruction: scale_vec::2X), which doubles
// the MACs per operand byte and per tensor-core cycle.  A stage then holds 256 K-elements.
// KIND 2 = dense BF16 operands (kind::f16, see mx_gemm_kernel): 64 K-elements per stage, no scales.
// BN = 384: the pair computes a 256 x 384 tile -- per stage one MMA with N = 256 (B rows 0..255 of the
// tile, 128 per CTA) and one with N = 128 (rows 256..383, 64 per CTA) -- which lowers the operand
// bytes each SM pulls from L2 per MAC from 1/128 to 1/153.6.  384 accumulator columns leave room for
// four stages of scale columns.
template <int KIND, int BN_>
struct Cfg2 {
  static_assert(BN_ == 256 || BN_ == 384, "tile width");
  static constexpr bool F4 = KIND == 1;
  static constexpr bool DENSE = KIND == 2;
  static constexpr int BN = BN_;
  static constexpr int kStages = BN == 384 ? (F4 ? 4 : 5) : 6;
  static constexpr int kBKe = F4 ? 256 : DENSE ? 64 : 128;  // K elements per stage (128-byte operand rows)
  static constexpr int kKChunks = F4 ? 2 : 1;           // 512-byte scale chunks (4 MX blocks) along K per stage
  static constexpr int kSfbGroups = BN / 128;           // 128-row scale chunks of B per K chunk
  static constexpr int kSfColsA = 4 * kKChunks;         // TMEM columns: this CTA's 128 rows of A
  static constexpr int kSfCols = kSfColsA + 4 * kSfbGroups * kKChunks;  // ... plus all BN rows of B
  static constexpr int kSfCol0 = BN;                    // single accumulator stage
  static constexpr uint32_t kBRows = BN / 2;            // rows of B this CTA stages
  static constexpr uint32_t kABytes = 128 * 128;        // this CTA's 128 rows of A, 128 bytes each
  static constexpr uint32_t kBBytes = kBRows * 128;
  static constexpr uint32_t kSfABytes = 512 * kKChunks;
  static constexpr uint32_t kSfBytes = kSfABytes + 512 * kSfbGroups * kKChunks;
  static constexpr uint32_t kOffA = 0;
  static constexpr uint32_t kOffB = kOffA + kStages * kABytes;
  static constexpr uint32_t kOffEpi = kOffB + kStages * kBBytes;
  static constexpr uint32_t kOffSf = kOffEpi + kEpiBytes;
  static constexpr uint32_t kOffBar = kOffSf + kStages * kSfBytes;
  static constexpr uint32_t kNumBars = 4 * kStages + 2;  // full, empty, scales ready, scales landed; accumulator x 2
  // Bytes used from the 1024-byte aligned base, and the request: up to 1024 bytes of slack for the
  // alignment, fewer where the budget is tight (the kernel checks that what it got suffices).
  static constexpr uint32_t kUsedBytes = kOffBar + kNumBars * 8 + 16;
  static constexpr uint32_t kSmemBytes = kUsedBytes + 1024 <= 232448 ? kUsedBytes + 1024 : 232448;
  static_assert(kUsedBytes <= 232448, "shared memory budget");
  static_assert(kSfCol0 + kStages * kSfCols <= kTmemCols, "tensor memory budget");
  // Convolution (mx_conv_pair_kernel): the A scale words of a K chunk are composed one trip round the
  // operand ring ahead of their use, into a ring of their own with twice as many slots, each with a
  // barrier in the leader (its own words + the peer's "mine have landed") and one in the peer.
  static constexpr uint32_t kConvSlots = 2 * kStages;
  static constexpr uint32_t kOffConvA = (kUsedBytes + 15u) & ~15u;
  static constexpr uint32_t kOffConvBar = kOffConvA + kConvSlots * 512;
  static constexpr uint32_t kConvUsedBytes = kOffConvBar + 2 * kConvSlots * 8;
  static constexpr uint32_t kConvSmemBytes = kConvUsedBytes + 1024;  // (checked where the kernel is defined)
};

// shared::cluster address of the same shared-memory offset in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}

__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, int x, int y,
                                                 int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_im2col_pair(uint32_t dst, const CUtensorMap* map, int c, int w, int h, int n,
                                                     uint32_t ow, uint32_t oh, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.im2col.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6], {%7, %8};"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c), "r"(w), "r"(h), "r"(n), "r"(bar),
        "h"((uint16_t)ow), "h"((uint16_t)oh) : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"((uint16_t)3) : "memory");
}
// The same, delivered to the leader CTA only.
__device__ __forceinline__ void tc_commit_leader(uint32_t bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"((uint16_t)1) : "memory");
}
__device__ __forceinline__ void tc_cp_scales_pair(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc,
                                            uint32_t idesc, uint32_t sfa_tmem, uint32_t sfb_tmem,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale.scale_vec::1X [%0], %1, %2, %3, [%4], [%5], p;\n\t"
      "}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(sfa_tmem), "r"(sfb_tmem),
        "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_mma_pair_f4(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc,
                                               uint32_t idesc, uint32_t sfa_tmem, uint32_t sfb_tmem,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::mxf4.block_scale.scale_vec::2X [%0], %1, %2, %3, [%4], [%5], p;\n\t"
      "}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(sfa_tmem), "r"(sfb_tmem),
        "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_mma_pair_dense(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc,
                                                  uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t"
      "}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// bar: shared::cluster address of a barrier (here: the leader CTA's, see leader_bar in the kernel)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// CONV: the implicit-GEMM convolution of mx_conv_kernel on the 256 x 256 pair tile (C % 128 == 0, so
// the codes of each CTA's 128 output pixels come through the im2col-mode map `tmap_a`); each CTA's
// scale-producer warp also composes the scale words of its 128 rows (four rows per lane).
// Work items of the pair kernel.  Tiles [0, split_from) are computed whole, pair p taking items p,
// p + P, ...; every tile from split_from on -- the last, less than half full round of the grid -- is
// dealt out as two items of 128 columns each (h = 1: columns 0..127 of the tile, h = 2: columns
// 128..255), so that twice as many pairs share that round and it takes about half a tile's time.
// A half item loads 64 rows of B per CTA (the second B map), issues MMAs with N = 128 into
// accumulator columns 0..127 and reads the B scales of its own 128-row group; the element order of
// every dot product is unchanged, so results do not depend on the split.
struct PairItem {
  uint32_t tile, h;
};
__device__ __forceinline__ PairItem pair_item(uint32_t i, uint32_t split_from) {
  if (i < split_from) return {i, 0u};
  const uint32_t j = i - split_from;
  return {split_from + (j >> 1), 1u + (j & 1u)};
}

template <int KIND, int BN_, bool CONV>
__device__ __forceinline__ void
pair_kernel_body(const CUtensorMap& tmap_a, const CUtensorMap& tmap_b, const CUtensorMap& tmap_b2,
                 const CUtensorMap& tmap_sa, const CUtensorMap& tmap_sb, const CUtensorMap& tmap_c,
                 uint32_t M, uint32_t N, uint32_t K, uint32_t idesc_base, uint32_t group_m,
                 uint32_t tx_bytes_pair, EpiArgs epi, uint32_t batch, long long spin_limit,
                 uint32_t drop_fill, const ConvGeom& cg, uint32_t split_from, uint32_t tx_bytes_half) {
  static_assert(!CONV || (KIND == 0 && BN_ == 256), "convolution runs on the block-scaled 256 x 256 tile");
  using cfg = Cfg2<KIND, BN_>;
  constexpr bool F4 = cfg::F4, DENSE = cfg::DENSE;
  constexpr int BN = cfg::BN;
  constexpr bool WIDE = BN == 384;
  constexpr int BKe = cfg::kBKe;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  if (smem_base - smem_u32(smem_raw) + (CONV ? cfg::kConvUsedBytes : cfg::kUsedBytes) > (CONV ? cfg::kConvSmemBytes : cfg::kSmemBytes)) {
    // the alignment cost more than the request left room for: give up before anything is set up
    // (uniform over the grid: every CTA sees the same offset)
    if (threadIdx.x == 0) atomicCAS(&g_gemm_status, 0u, (unsigned int)ST_SMEM_ALIGN);
    return;
  }
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar0 = smem_base + cfg::kOffBar;
  auto full_bar = [&](uint32_t s) { return bar0 + 8 * s; };
  auto empty_bar = [&](uint32_t s) { return bar0 + 8 * (cfg::kStages + s); };
  const uint32_t acc_full_bar = bar0 + 8 * (2 * cfg::kStages);
  const uint32_t acc_empty_bar = bar0 + 8 * (2 * cfg::kStages + 1);
  auto sf_ready_bar = [&](uint32_t s) { return bar0 + 8 * (2 * cfg::kStages + 2 + s); };
  auto sf_full_bar = [&](uint32_t s) { return bar0 + 8 * (3 * cfg::kStages + 2 + s); };
  auto conv_a_slot = [&](uint32_t j) { return smem_base + cfg::kOffConvA + 512u * j; };
  auto a_ok_bar = [&](uint32_t j) { return smem_base + cfg::kOffConvBar + 8u * j; };                  // used in the leader
  auto asf_bar = [&](uint32_t j) { return smem_base + cfg::kOffConvBar + 8u * (cfg::kConvSlots + j); };  // used in the peer
  volatile uint32_t* tmem_slot =
      reinterpret_cast<volatile uint32_t*>(smem_gen + cfg::kOffBar + cfg::kNumBars * 8);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  // the leader CTA's copy of one of the barriers above, as a shared::cluster address (both CTAs
  // use the same shared-memory layout, so it is the mapped base plus the barrier's offset)
  const uint32_t bar0_leader = map_to_cta(bar0, 0);
  auto leader_bar = [&](uint32_t local_bar) { return bar0_leader + (local_bar - bar0); };

  uint32_t rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  const uint32_t tiles_m = (M + 255) / 256, tiles_n = (N + BN - 1) / BN;
  // items, not tiles, are what the roles below walk (see pair_item); without a split the two are the same
  const uint32_t num_tiles = split_from + 2u * (batch * tiles_m * tiles_n - split_from);
  const uint32_t k_chunks = (K + BKe - 1) / BKe;  // a K tail is zero-filled by the copies

  if (threadIdx.x == 0) {
    for (uint32_t s = 0; s < cfg::kStages; ++s) {
      mbar_init(full_bar(s), 1);   // used in the leader only: its producer's arrive + all bytes
      mbar_init(empty_bar(s), 1);  // one tcgen05.commit per use, delivered to both CTAs
      mbar_init(sf_ready_bar(s), 1);  // used in the leader only: the copier's tcgen05.commit
      // used in the leader only: the scale producer's arrive + scale bytes
      mbar_init(sf_full_bar(s), 1);
    }
    mbar_init(acc_full_bar, 1);
    mbar_init(acc_empty_bar, 16);  // eight epilogue warps in each CTA (the leader's barrier is used)
    if (CONV) {
      for (uint32_t j = 0; j < cfg::kConvSlots; ++j) {
        mbar_init(a_ok_bar(j), 33);  // the 32 lanes of the leader's scale-producer warp + the peer's relay
        mbar_init(asf_bar(j), 32);   // the 32 lanes of the peer's scale-producer warp
      }
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_a)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_b)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_sa)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_sb)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_c)) : "memory");
  }
  if (warp == 1) {  // the same warp in both CTAs: the allocation is collective over the pair
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))), "r"((uint32_t)kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync();  // the peer's barriers exist before anything is signalled remotely
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  asm volatile("griddepcontrol.wait;" ::: "memory");  // as in mx_gemm_kernel

  if (warp == 0) {
    // ------------------------- TMA producer (both CTAs) -------------------------
    // Operand tiles only: the scale chunks have a producer warp of their own (below).  The whole
    // warp runs the loop converged and one elected lane issues the copies (see elect_one).
    // drop_fill: see the operand producer of mx_gemm_kernel (both CTAs leave out the same fill).
    uint32_t stage = 0, phase = 0, fill = 0;
    bool ok = true;
    for (uint32_t t = pair; t < num_tiles && ok; t += num_pairs) {
      const PairItem it = pair_item(t, split_from);
      const TileCoord tc = tile_coord(it.tile, tiles_m, tiles_n, group_m);
      // this CTA's 128 rows of A and its rows of B: rows 128 rank .. of the tile and, for the wide
      // tile, rows 256 + 64 rank .. (B rows may lie past N on a ragged tile: zero fill or the next
      // matrix of a batch; their columns are not stored); a half item: rows 128 (h - 1) + 64 rank ..
      const int cy_a = (int)((tc.b * tiles_m + tc.tm) * 256 + rank * 128);
      const int cy_b = (int)(tc.b * N + tc.tn * BN + rank * 128);
      const int cy_b2 = it.h ? (int)(tc.b * N + tc.tn * BN + (it.h - 1u) * 128u + rank * 64)
                             : (int)(tc.b * N + tc.tn * BN + 256 + rank * 64);
      // CONV: where tap (0, 0) of the first of this CTA's 128 output pixels reads
      int cv_w = 0, cv_h = 0, cv_n = 0;
      if (CONV) {
        const uint32_t m0 = tc.tm * 256 + rank * 128, n0 = fastdiv(m0, cg.d_howo), rem = m0 - n0 * (cg.Ho * cg.Wo);
        const uint32_t ho = fastdiv(rem, cg.d_wo), wo = rem - ho * cg.Wo;
        cv_n = (int)n0;
        cv_h = (int)ho * cg.stride_h - cg.pad_h;
        cv_w = (int)wo * cg.stride_w - cg.pad_w;
      }
      for (uint32_t kc = 0; kc < k_chunks; ++kc) {
        ok = __all_sync(0xffffffffu, mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, spin_limit));
        if (!ok) {
          raise_abort(abort_flag, ST_PRODUCER_WAIT);
          break;
        }
        if (fill++ != drop_fill && elect_one()) {
          const uint32_t fb = leader_bar(full_bar(stage));
          if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), it.h ? tx_bytes_half : tx_bytes_pair);
          const int cx = (int)(kc * BKe);
          if (CONV) {  // the stage's K chunk = 128 channels of one filter tap
            const uint32_t tap = fastdiv(kc * 4, cg.d_cb), cblk = kc * 4 - tap * cg.cb;
            const uint32_t ti = fastdiv(tap, cg.d_kw), tj = tap - ti * cg.kw;
            tma_load_im2col_pair(smem_base + cfg::kOffA + stage * cfg::kABytes, &tmap_a, (int)(cblk * 32u), cv_w, cv_h,
                                 cv_n, tj * (uint32_t)cg.dil_w, ti * (uint32_t)cg.dil_h, fb);
          } else {
            tma_load_3d_pair(smem_base + cfg::kOffA + stage * cfg::kABytes, &tmap_a, cx, cy_a, 0, fb);
          }
          if (it.h)  // 64 rows of B at the start of the stage's B area
            tma_load_3d_pair(smem_base + cfg::kOffB + stage * cfg::kBBytes, &tmap_b2, cx, cy_b2, 0, fb);
          else
            tma_load_3d_pair(smem_base + cfg::kOffB + stage * cfg::kBBytes, &tmap_b, cx, cy_b, 0, fb);
          if (WIDE)
            tma_load_3d_pair(smem_base + cfg::kOffB + stage * cfg::kBBytes + 128u * 128u, &tmap_b2, cx, cy_b2, 0, fb);
        }
        __syncwarp();
        if (++stage == cfg::kStages) { stage = 0; phase ^= 1u; }
      }
    }
    if (!ok) {  // let copies that are still in flight land before the CTA goes away
      const long long t0 = clock64();
      while (clock64() - t0 < 2000000LL) {}
    }
  } else if (warp == 1) {
    // --------------------------- MMA issuer (leader) ---------------------------
    // the warp runs converged; one elected lane issues a stage's MMAs and the commit
    if (rank == 0) {
      uint32_t stage = 0, phase = 0, acc_phase = 0;
      bool ok = true;
      for (uint32_t t = pair; t < num_tiles && ok; t += num_pairs) {
        const uint32_t hsel = pair_item(t, split_from).h;
        if (!__all_sync(0xffffffffu, mbar_wait(acc_empty_bar, acc_phase ^ 1u, abort_flag, 4 * spin_limit))) {
          raise_abort(abort_flag, ST_MMA_WAIT_ACC);
          break;
        }
        tc_fence_after();
        for (uint32_t kc = 0; kc < k_chunks; ++kc) {
          // scales in tensor memory, then the operands
          ok = __all_sync(0xffffffffu, (DENSE || mbar_wait(sf_ready_bar(stage), phase, abort_flag, spin_limit)) &&
                                           mbar_wait(full_bar(stage), phase, abort_flag, spin_limit));
          if (!ok) {
            raise_abort(abort_flag, ST_MMA_WAIT_FULL);
            break;
          }
          tc_fence_after();
          const uint32_t sf_tmem = tmem_base + cfg::kSfCol0 + stage * cfg::kSfCols;
          const uint64_t adesc = operand_desc(smem_base + cfg::kOffA + stage * cfg::kABytes);
          const uint64_t bdesc = operand_desc(smem_base + cfg::kOffB + stage * cfg::kBBytes);
          // wide tile: columns 256..383 come from a second MMA with N = 128 on the B rows staged
          // behind the first 128 (64 per CTA); its B scales are the third 128-row group
          const uint64_t bdesc2 = operand_desc(smem_base + cfg::kOffB + stage * cfg::kBBytes + 128u * 128u);
          const uint32_t idesc2_base = (idesc_base & ~(0x3Fu << 17)) | ((uint32_t)(128 >> 3) << 17);
          constexpr uint32_t kSfbStep = 4 * cfg::kSfbGroups;  // B scale columns per K chunk
          // a half item: N = 128, the B scales of its own 128-row group (4 columns further for h = 2)
          const uint32_t idesc1 = hsel ? idesc2_base : idesc_base;
          const uint32_t sfb_h = hsel ? 4u * (hsel - 1u) : 0u;
          if (elect_one()) {
#pragma unroll
          for (uint32_t k = 0; k < 4; ++k) {  // every MMA advances 32 bytes along the 128-byte rows
            const uint32_t acc_flag = (kc | k) != 0 ? 1u : 0u;
            if (DENSE) {
              tc_mma_pair_dense(tmem_base, adesc + 2 * k, bdesc + 2 * k, idesc1, acc_flag);
              if (WIDE) tc_mma_pair_dense(tmem_base + 256, adesc + 2 * k, bdesc2 + 2 * k, idesc2_base, acc_flag);
            } else if (F4) {
              // K = 64: blocks 2k and 2k+1 of the stage = bytes (2k % 4, +1) of K chunk k / 2
              const uint32_t sf_id = 2 * (k & 1);
              const uint32_t sel = (sf_id << 4) | (sf_id << 29);
              const uint32_t sfa = sf_tmem + 4 * (k >> 1), sfb = sf_tmem + cfg::kSfColsA + kSfbStep * (k >> 1) + sfb_h;
              tc_mma_pair_f4(tmem_base, adesc + 2 * k, bdesc + 2 * k, idesc1 | sel, sfa, sfb, acc_flag);
              if (WIDE)
                tc_mma_pair_f4(tmem_base + 256, adesc + 2 * k, bdesc2 + 2 * k, idesc2_base | sel, sfa, sfb + 8,
                               acc_flag);
            } else {
              const uint32_t sel = (k << 4) | (k << 29);  // byte k of the scale columns
              const uint32_t sfb = sf_tmem + cfg::kSfColsA + sfb_h;
              tc_mma_pair(tmem_base, adesc + 2 * k, bdesc + 2 * k, idesc1 | sel, sf_tmem, sfb, acc_flag);
              if (WIDE)
                tc_mma_pair(tmem_base + 256, adesc + 2 * k, bdesc2 + 2 * k, idesc2_base | sel, sf_tmem, sfb + 8,
                            acc_flag);
            }
          }
          tc_commit_pair(empty_bar(stage));
          }
          __syncwarp();
          if (++stage == cfg::kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok && elect_one()) tc_commit_pair(acc_full_bar);
        __syncwarp();
        acc_phase ^= 1u;
      }
    }
  } else if (warp == 10) {
    // --------------------------- scale copier (leader) ---------------------------
    if constexpr (!DENSE) {
      if (rank == 0) {
        uint32_t stage = 0, phase = 0, conv_chunk = 0;
        bool ok = true;
        for (uint32_t t = pair; t < num_tiles && ok; t += num_pairs) {
          for (uint32_t kc = 0; kc < k_chunks; ++kc) {
            const uint32_t aslot = conv_chunk % cfg::kConvSlots, aparity = (conv_chunk / cfg::kConvSlots) & 1u;
            ok = __all_sync(0xffffffffu, mbar_wait(sf_full_bar(stage), phase, abort_flag, spin_limit) &&
                                             (!CONV || mbar_wait(a_ok_bar(aslot), aparity, abort_flag, spin_limit)));
            if (!ok) {
              raise_abort(abort_flag, ST_SCALE_WAIT);
              break;
            }
            // CONV: the A scale words were written by ordinary copies (the peer fenced its own before it arrived)
            if (CONV) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            ++conv_chunk;
            tc_fence_after();
            const uint32_t sf_smem = smem_base + cfg::kOffSf + stage * cfg::kSfBytes;
            const uint32_t sf_tmem = tmem_base + cfg::kSfCol0 + stage * cfg::kSfCols;
            // Each CTA copies from its own shared memory to its own tensor memory.  A: K chunk c at
            // columns 4c.  B: the box is [row group][K chunk], and the MMA wants the columns of one
            // K chunk together: group g of G, chunk c -> 4 G c + 4g.
            if (elect_one()) {
#pragma unroll
              for (uint32_t c = 0; c < cfg::kKChunks; ++c) {
                tc_cp_scales_pair(sf_tmem + 4 * c, scale_desc(CONV ? conv_a_slot(aslot) : sf_smem + 512 * c));
#pragma unroll
                for (uint32_t g = 0; g < cfg::kSfbGroups; ++g)
                  tc_cp_scales_pair(sf_tmem + cfg::kSfColsA + 4 * cfg::kSfbGroups * c + 4 * g,
                                    scale_desc(sf_smem + cfg::kSfABytes + 512 * (g * cfg::kKChunks + c)));
              }
              tc_commit_leader(sf_ready_bar(stage));  // arrives when the copies have completed in both CTAs
            }
            __syncwarp();
            if (++stage == cfg::kStages) { stage = 0; phase ^= 1u; }
          }
        }
      } else if (CONV) {
        // the peer CTA: pass "my A scale words of chunk g are in my shared memory (and visible to
        // the tensor core's proxy)" on to the leader's barrier of that slot; this warp has no copies
        // of its own in flight, so its fence and its arrival wait for nothing
        uint32_t g = 0;
        bool ok = true;
        for (uint32_t t = pair; t < num_tiles && ok; t += num_pairs) {
          for (uint32_t kc = 0; kc < k_chunks; ++kc, ++g) {
            const uint32_t j = g % cfg::kConvSlots;
            ok = __all_sync(0xffffffffu, mbar_wait(asf_bar(j), (g / cfg::kConvSlots) & 1u, abort_flag, spin_limit));
            if (!ok) {
              raise_abort(abort_flag, ST_SCALE_WAIT);
              break;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            // An arrival with the default semantics: the words stay in this CTA's shared memory and
            // the fence above has made them visible to this SM's tensor-core proxy, which is the only
            // reader; nothing is published to the other CTA's threads.  (A release at cluster scope
            // here took ~0.8 us per arrival and set the pace of the whole kernel: 92 against 61 us.)
            if (lane == 0) mbar_arrive_cluster(map_to_cta(a_ok_bar(j), 0));
          }
        }
      }
    }
  } else if (warp == 11) {
    // ------------------------ scale producer (both CTAs) ------------------------
    // This CTA's A scales and the B scales of all BN columns; both copies complete on the leader's
    // per-stage "scales landed" barrier, which the leader arms.  A stage's scale buffer and scale
    // columns are free when the stage is (the MMAs that read them have completed).
    if constexpr (!DENSE) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      // CONV: the A scale words.  Lane l copies the words of rows l, l + 32, l + 64, l + 96 of this
      // CTA's 128 output pixels from the activation's scale tensor, asynchronously, into the slot of
      // the chunk's running number; a cursor walks the CTA's chunks one ring round ahead of the loop
      // below (so a word has a whole round to arrive, and the hop through the peer's relay is hidden).
      uint32_t g_tile = pair, g_kc = 0, g_num = 0;   // the cursor: tile, K chunk, running chunk number
      int32_t cvh[4] = {0, 0, 0, 0}, cvw[4] = {0, 0, 0, 0};
      uint32_t cvp[4] = {0, 0, 0, 0};  // first pixel of the row's image; 0xFFFFFFFF: row past M
      auto conv_rows = [&]() {  // geometry of the cursor's tile
        const TileCoord gc = tile_coord(g_tile, tiles_m, tiles_n, group_m);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t m = gc.tm * 256 + rank * 128 + lane + 32 * j;
          const uint32_t n0 = fastdiv(m, cg.d_howo), rem = m - n0 * (cg.Ho * cg.Wo);
          const uint32_t ho = fastdiv(rem, cg.d_wo), wo = rem - ho * cg.Wo;
          cvh[j] = (int32_t)ho * cg.stride_h - cg.pad_h;
          cvw[j] = (int32_t)wo * cg.stride_w - cg.pad_w;
          cvp[j] = m < cg.M ? n0 * cg.H * cg.W : 0xFFFFFFFFu;
        }
      };
      auto conv_gather = [&]() {  // the cursor's chunk, then move the cursor on
        if (g_tile >= num_tiles) return;
        const uint32_t slot = g_num % cfg::kConvSlots;
        // the K chunk is 128 channels of one filter tap: one aligned word of scales per row
        const uint32_t tap = fastdiv(g_kc * 4, cg.d_cb), cblk = g_kc * 4 - tap * cg.cb;
        const uint32_t ti = fastdiv(tap, cg.d_kw), tj = tap - ti * cg.kw;
        const int32_t dh = (int32_t)ti * cg.dil_h, dw = (int32_t)tj * cg.dil_w;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int32_t hi = cvh[j] + dh, wi = cvw[j] + dw;
          const bool live = cvp[j] != 0xFFFFFFFFu && hi >= 0 && hi < (int32_t)cg.H && wi >= 0 && wi < (int32_t)cg.W;
          const uint32_t px = live ? cvp[j] + (uint32_t)hi * cg.W + (uint32_t)wi : 0u;
          const size_t so = cg.x_layout == MX_SCALES_LINEAR ? (size_t)px * cg.cb + cblk
                                                            : scale_offset<MX_SCALES_SWIZZLED>(px, cblk, cg.cb);
          // row r = lane + 32 j of the chunk lives at byte (r % 32) * 16 + (r / 32) * 4
          cp_async_4(conv_a_slot(slot) + lane * 16u + (uint32_t)j * 4u, cg.x_scales + (live ? so : 0), live ? 4u : 0u);
        }
        cp_async_arrive(rank == 0 ? a_ok_bar(slot) : asf_bar(slot));
        ++g_num;
        if (++g_kc == k_chunks) {
          g_kc = 0;
          g_tile += num_pairs;
          if (g_tile < num_tiles) conv_rows();
        }
      };
      if (CONV && g_tile < num_tiles) {
        conv_rows();
        for (uint32_t i = 0; i < (uint32_t)cfg::kStages; ++i) conv_gather();  // the first round's chunks at once
      }
      for (uint32_t t = pair; t < num_tiles && ok; t += num_pairs) {
        // (a half item fetches the B scales of both 128-row groups of its tile; its MMAs read one)
        const TileCoord tc = tile_coord(pair_item(t, split_from).tile, tiles_m, tiles_n, group_m);
        const int cz_a = (int)((tc.b * tiles_m + tc.tm) * 2 + rank);
        const int cz_b = (int)(tc.b * (N / 128) + tc.tn * cfg::kSfbGroups);
        for (uint32_t kc = 0; kc < k_chunks; ++kc) {
          ok = __all_sync(0xffffffffu, mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, spin_limit));
          if (!ok) {
            raise_abort(abort_flag, ST_PRODUCER_WAIT);
            break;
          }
          if (elect_one()) {
            const uint32_t fb = leader_bar(sf_full_bar(stage));
            if (rank == 0) mbar_arrive_expect_tx(sf_full_bar(stage), 2u * (CONV ? cfg::kSfBytes - cfg::kSfABytes : cfg::kSfBytes));
            const uint32_t dst = smem_base + cfg::kOffSf + stage * cfg::kSfBytes;
            if (!CONV) tma_load_3d_pair(dst, &tmap_sa, 0, (int)(kc * cfg::kKChunks), cz_a, fb);
            tma_load_3d_pair(dst + cfg::kSfABytes, &tmap_sb, 0, (int)(kc * cfg::kKChunks), cz_b, fb);
          }
          __syncwarp();
          // the stage just freed belonged to the chunk one ring round back, and so did the A-scale
          // slot that the chunk one round AHEAD will use: compose that chunk's words now
          if (CONV) conv_gather();
          if (++stage == cfg::kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (CONV) asm volatile("cp.async.wait_all;" ::: "memory");
      if (!ok) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
      }
    }
  } else {
    // ---------------------------- epilogue (both CTAs) ----------------------------
    const uint32_t quarter = warp & 3u;
    const uint32_t half = (warp - 2u) >> 2;
    constexpr uint32_t kHalf = BN / 2, kLoads = kHalf / 32;
    uint32_t acc_phase = 0;
    for (uint32_t t = pair; t < num_tiles; t += num_pairs) {
      const PairItem it = pair_item(t, split_from);
      const TileCoord tc = tile_coord(it.tile, tiles_m, tiles_n, group_m);
      if (!mbar_wait(acc_full_bar, acc_phase, abort_flag, 4 * spin_limit)) {
        if (lane == 0) raise_abort(abort_flag, ST_EPILOGUE_WAIT);
        break;
      }
      tc_fence_after();
      const uint32_t row0 = (tc.b * tiles_m + tc.tm) * 256 + rank * 128 + quarter * 32;
      if constexpr (WIDE) {
        // 192 columns per warp in two passes of 96 (registers); the accumulator is handed back
        // after the second pass's loads.  The quantizing epilogue is not offered at this width.
        constexpr uint32_t kPass = 96, kPassLoads = 3;
#pragma unroll 1
        for (uint32_t pass = 0; pass < 2; ++pass) {
          const uint32_t cofs = half * kHalf + pass * kPass;
          const uint32_t taddr = tmem_base + ((quarter * 32u) << 16) + cofs;
          const uint32_t col0 = tc.tn * BN + cofs;
          // nothing to store for a warp whose rows or columns lie past the matrix
          const uint32_t valid_cols = (col0 < N && row0 < batch * M) ? min(kPass, N - col0) : 0u;
          uint32_t r[kPassLoads][32];
#pragma unroll
          for (uint32_t j = 0; j < kPassLoads; ++j) tc_ld32(taddr + 32 * j, r[j]);
          tc_wait_ld();
          if (pass == 1) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(leader_bar(acc_empty_bar));
          }
          store_rows<kPassLoads>(r, smem_base + cfg::kOffEpi + (warp - 2u) * kEpiBufs * kEpiChunkBytes, &tmap_c,
                                 (int)col0, (int)row0, valid_cols, lane, epi.mode);
        }
      } else {
        const uint32_t taddr = tmem_base + ((quarter * 32u) << 16) + half * kHalf;
        // a half item: its 128 columns are accumulator columns 0..127, read out by the first four
        // warps; the other four only hand the accumulator back
        const uint32_t col0 = it.h ? tc.tn * BN + (it.h - 1u) * 128u : tc.tn * BN + half * kHalf;
        // nothing to store for a warp whose rows or columns lie past the matrix
        const uint32_t valid_cols = (col0 < N && row0 < batch * M && !(it.h && half)) ? min(kHalf, N - col0) : 0u;
        uint32_t r[kLoads][32];
#pragma unroll
        for (uint32_t j = 0; j < kLoads; ++j) tc_ld32(taddr + 32 * j, r[j]);
        tc_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(leader_bar(acc_empty_bar));  // accumulator rows of this CTA are in registers
        if (epi.mode == 2) {
          if (valid_cols) store_mx_rows<kLoads>(r, epi, row0 + lane, col0, N);
        } else {
          store_rows<kLoads>(r, smem_base + cfg::kOffEpi + (warp - 2u) * kEpiBufs * kEpiChunkBytes, &tmap_c,
                             (int)col0, (int)row0, valid_cols, lane, epi.mode);
        }
      }
      acc_phase ^= 1u;
    }
    if (lane == 0) bulk_wait_read<0>();  // the stores have left shared memory; the kernel's end orders the writes
  }

  // common exit: both CTAs of the pair leave together, then the pair's tensor memory is freed
  tc_fence_before();
  __syncthreads();
  cluster_sync();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"((uint32_t)kTmemCols) : "memory");
  }
}

template <int KIND, int BN_>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
mx_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                    const __grid_constant__ CUtensorMap tmap_b2,
                    const __grid_constant__ CUtensorMap tmap_sa, const __grid_constant__ CUtensorMap tmap_sb,
                    const __grid_constant__ CUtensorMap tmap_c, uint32_t M, uint32_t N, uint32_t K,
                    uint32_t idesc_base, uint32_t group_m, uint32_t tx_bytes_pair, EpiArgs epi,
                    uint32_t batch, long long spin_limit, uint32_t drop_fill, uint32_t split_from,
                    uint32_t tx_bytes_half) {
  const ConvGeom none = {};
  pair_kernel_body<KIND, BN_, false>(tmap_a, tmap_b, tmap_b2, tmap_sa, tmap_sb, tmap_c, M, N, K, idesc_base, group_m,
                                     tx_bytes_pair, epi, batch, spin_limit, drop_fill, none, split_from, tx_bytes_half);
}

static_assert(Cfg2<0, 256>::kConvSmemBytes <= 232448, "shared memory budget of the convolution kernel");
// Implicit-GEMM convolution on the pair tile (tmap_x: the im2col-mode map over the activation's codes).
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
mx_conv_pair_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_b,
                    const __grid_constant__ CUtensorMap tmap_sb, const __grid_constant__ CUtensorMap tmap_c,
                    uint32_t M, uint32_t N, uint32_t K, uint32_t idesc_base, uint32_t group_m,
                    uint32_t tx_bytes_pair, EpiArgs epi, long long spin_limit, const __grid_constant__ ConvGeom cg) {
  // (no split of the last round: every tile whole)
  pair_kernel_body<0, 256, true>(tmap_x, tmap_b, tmap_b, tmap_sb, tmap_sb, tmap_c, M, N, K, idesc_base, group_m,
                                 tx_bytes_pair, epi, 1u, spin_limit, kNoDrop, cg, ((M + 255) / 256) * ((N + 255) / 256), 0u);
}

// ---- host side ---------------------------------------------------------------

int fmt_bits(int f) { return f == MX_E2M1 ? 4 : ((f == MX_E3M2 || f == MX_E2M3) ? 6 : 8); }

// Format field of the instruction descriptor.
uint32_t mma_fmt_code(int f) {
  switch (f) {
    case MX_E4M3: return 0;
    case MX_E5M2: return 1;
    case MX_E2M3: return 3;
    case MX_E3M2: return 4;
    default: return 5;  // MX_E2M1
  }
}

// Tensor map of a packed K-major operand [rows x K]: box = 128 elements x box_rows,
// 128-byte swizzle.  FP6 / FP4 use the packed types that expand to 16-byte containers.
bool make_operand_map(EncodeTiledFn fn, CUtensorMap* map, const void* ptr, int fmt, uint64_t rows,
                      uint64_t K, uint32_t box_rows) {
  const int bits = fmt_bits(fmt);
  const CUtensorMapDataType dt = bits == 8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                                 : bits == 6 ? CU_TENSOR_MAP_DATA_TYPE_16U6_ALIGN16B
                                             : CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B;
  const cuuint64_t pitch = K * (uint64_t)bits / 8;
  const cuuint64_t dims[3] = {K, rows, 1};
  const cuuint64_t strides[2] = {pitch, pitch * rows};
  const cuuint32_t box[3] = {(cuuint32_t)BK, box_rows, 1};
  return encode_cached(fn, map, dt, 3, ptr, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B,
                       CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
}

// Tensor map of a dense BF16 K-major operand [rows x K]: box = 64 elements (128 bytes) x box_rows.
bool make_dense_map(EncodeTiledFn fn, CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t K,
                    uint32_t box_rows) {
  const cuuint64_t dims[3] = {K, rows, 1};
  const cuuint64_t strides[2] = {K * 2, K * 2 * rows};
  const cuuint32_t box[3] = {64, box_rows, 1};
  return encode_cached(fn, map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, ptr, dims, strides, box,
                       CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
}

// Tensor map over a swizzled scale tensor seen as [row groups of 128][K chunks][128 words]:
// one 512-byte chunk per (row group, K chunk); the box takes `groups` consecutive row groups.
bool make_scale_map(EncodeTiledFn fn, CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t K,
                    uint32_t groups) {
  const uint64_t k_chunks = (K + BK - 1) / BK;  // the swizzled layout pads K to whole chunks, rows to 128
  const cuuint64_t dims[3] = {128, k_chunks, (rows + 127) / 128};
  const cuuint64_t strides[2] = {512, 512 * k_chunks};
  const cuuint32_t box[3] = {128, 1, groups};
  return encode_cached(fn, map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, ptr, dims, strides, box,
                       CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
}

// Tensor map of the output [M x N] (FP32 or BF16): box = 64 bytes of columns x 32 rows in the
// 64-byte swizzle the epilogue writes its staging chunks in.
bool make_c_map(EncodeTiledFn fn, CUtensorMap* map, void* C, uint64_t M, uint64_t N, bool bf16) {
  const cuuint64_t dims[2] = {N, M};
  const cuuint64_t strides[1] = {N * (bf16 ? 2u : 4u)};
  const cuuint32_t box[2] = {bf16 ? 32u : kEpiChunkCols, 32};
  return encode_cached(fn, map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, C,
                       dims, strides, box, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE);
}

// The output map the kernels take.  A quantizing epilogue writes with plain stores and never uses
// it; it still gets a valid map (over the code tensor) because the kernel prefetches the descriptor.
bool make_out_map(EncodeTiledFn fn, CUtensorMap* map, const GemmArgs& a) {
  if (a.q_elems) return make_c_map(fn, map, a.q_elems, (uint64_t)(a.batch * a.M), (uint64_t)a.N / 4, true);
  return make_c_map(fn, map, a.C, (uint64_t)(a.batch * a.M), (uint64_t)a.N, a.c_bf16 != 0);
}

// The GEMM kernels are launched with programmatic stream serialization like the streaming kernels:
// their set-up (barriers, tensor-memory allocation, descriptor fetch) overlaps the tail of the kernel
// before them -- 14.0 -> 12.5 us per launch for back-to-back 256 x 256 x 1024 products, 57.8 -> 56.1
// us for 4096^3, nothing lost on the largest ones (when the kernels still announced their own
// dependents early, chains of large products were 3 % slower with it; they no longer do).

long long wait_budget(const GemmArgs& a) { return a.wait_cycles > 0 ? (long long)a.wait_cycles : kSpinLimit; }
uint32_t drop_fill(const GemmArgs& a) { return a.drop_fill >= 0 ? (uint32_t)a.drop_fill : kNoDrop; }

EpiArgs epi_args(const GemmArgs& a) {
  EpiArgs e;
  e.mode = a.q_elems ? 2u : (a.c_bf16 ? 1u : 0u);
  e.fmt = (uint32_t)a.q_fmt;
  e.sticky = a.q_round == MX_RHAZ ? 1u : 0u;
  e.elems = (uint8_t*)a.q_elems;
  e.scales = a.q_scales;
  return e;
}

template <int BN, bool DENSE>
cudaError_t launch_bn(const GemmArgs& a, const CUtensorMap& ma, const CUtensorMap& mb,
                      uint32_t idesc_base) {
  CUtensorMap mc, msa, msb;
  EncodeTiledFn fn = encode_fn_cached();
  if (!make_out_map(fn, &mc, a)) return cudaErrorInvalidValue;
  if (DENSE) {
    msa = ma;  // the dense kernel takes no scales; the parameters still hold valid descriptors
    msb = mb;
  } else if (!make_scale_map(fn, &msa, a.sA, (uint64_t)(a.batch * a.M), (uint64_t)a.K, 1) ||
             !make_scale_map(fn, &msb, a.sB, (uint64_t)(a.batch * a.N), (uint64_t)a.K, Cfg<BN>::kSfbChunks)) {
    return cudaErrorInvalidValue;
  }
  using cfg = Cfg<BN>;
  static bool attr_set[64] = {false};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    e = cudaFuncSetAttribute(mx_gemm_kernel<BN, DENSE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)cfg::kSmemBytes);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  const uint32_t tiles = (uint32_t)a.batch * (uint32_t)((a.M + BM - 1) / BM) * (uint32_t)((a.N + BN - 1) / BN);
  const uint32_t grid = tiles < (uint32_t)a.sm_count ? tiles : (uint32_t)a.sm_count;
  const uint32_t group_m = 16;
  // Bytes the operand copies report to a stage's mbarrier: the tensor-map copies count the packed
  // source bytes (bits/8 per element), not the expanded shared-memory footprint.  The scale chunks
  // complete on a barrier of their own.
  const uint32_t tx_bytes =
      DENSE ? (uint32_t)(BM + BN) * 128u
            : (uint32_t)(BM * BK * fmt_bits(a.fmtA) / 8 + BN * BK * fmt_bits(a.fmtB) / 8);
  return launch_pdl(mx_gemm_kernel<BN, DENSE>, dim3(grid), dim3(kThreads), cfg::kSmemBytes, a.stream,
                    ma, mb, msa, msb, mc, (uint32_t)a.M, (uint32_t)a.N, (uint32_t)a.K,
                    idesc_base | ((uint32_t)(BN >> 3) << 17), group_m, tx_bytes, epi_args(a),
                    (uint32_t)a.batch, wait_budget(a), drop_fill(a));
}

// Dense FP4 operand map for kind::mxf4: two codes per byte in shared memory as in global memory.
bool make_f4_map(EncodeTiledFn fn, CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t K,
                 uint32_t box_rows = 128) {
  const cuuint64_t pitch = K / 2;
  const cuuint64_t dims[3] = {K, rows, 1};
  const cuuint64_t strides[2] = {pitch, pitch * rows};
  const cuuint32_t box[3] = {256, box_rows, 1};
  return encode_cached(fn, map, CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN8B, 3, ptr, dims, strides, box,
                       CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
}

// Scale map whose box also spans `kchunks` K chunks: [row groups][K chunks][128 words].
bool make_scale_map_k(EncodeTiledFn fn, CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t K,
                      uint32_t groups, uint32_t kchunks) {
  const uint64_t k_chunks = (K + BK - 1) / BK;  // the swizzled layout pads K to whole chunks, rows to 128
  const cuuint64_t dims[3] = {128, k_chunks, (rows + 127) / 128};
  const cuuint64_t strides[2] = {512, 512 * k_chunks};
  const cuuint32_t box[3] = {128, kchunks, groups};
  return encode_cached(fn, map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, ptr, dims, strides, box,
                       CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
}

template <int KIND, int BN>
cudaError_t launch_pair(const GemmArgs& a, EncodeTiledFn fn) {
  using cfg = Cfg2<KIND, BN>;
  constexpr bool F4 = cfg::F4, DENSE = cfg::DENSE, WIDE = BN == 384;
  // rows of B a CTA takes with its second copy (wide tile): 64; the map is unused otherwise
  constexpr uint32_t kB2Rows = 64;  // (also what a CTA loads for a half item, see pair_item)
  const uint64_t rows_a = (uint64_t)(a.batch * a.M), rows_b = (uint64_t)(a.batch * a.N), K = (uint64_t)a.K;
  CUtensorMap ma, mb, mb2, msa, msb, mc;
  bool ok = make_out_map(fn, &mc, a);
  if (DENSE) {
    ok = ok && make_dense_map(fn, &ma, a.A, rows_a, K, 128) && make_dense_map(fn, &mb, a.B, rows_b, K, 128) &&
         make_dense_map(fn, &mb2, a.B, rows_b, K, kB2Rows);
    msa = ma;  // no scales: valid descriptors the kernel never uses
    msb = mb;
  } else {
    ok = ok && make_scale_map_k(fn, &msa, a.sA, rows_a, K, 1, cfg::kKChunks) &&
         make_scale_map_k(fn, &msb, a.sB, rows_b, K, cfg::kSfbGroups, cfg::kKChunks);
    if (F4)
      ok = ok && make_f4_map(fn, &ma, a.A, rows_a, K) && make_f4_map(fn, &mb, a.B, rows_b, K) &&
           make_f4_map(fn, &mb2, a.B, rows_b, K, kB2Rows);
    else
      ok = ok && make_operand_map(fn, &ma, a.A, a.fmtA, rows_a, K, 128) &&
           make_operand_map(fn, &mb, a.B, a.fmtB, rows_b, K, 128) &&
           make_operand_map(fn, &mb2, a.B, a.fmtB, rows_b, K, kB2Rows);
  }
  if (!ok) return cudaErrorInvalidValue;
  static bool attr_set[64] = {false};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    e = cudaFuncSetAttribute(mx_gemm_pair_kernel<KIND, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)cfg::kSmemBytes);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  const uint32_t tiles = (uint32_t)a.batch * (uint32_t)((a.M + 255) / 256) * (uint32_t)((a.N + BN - 1) / BN);
  // A last round that would occupy at most half of the pairs is dealt out in halves of 128 columns
  // (4096^3: 256 tiles on 74 pairs = three rounds + 34 tiles -> 68 half items: 57.3 -> 55.0 us; a half
  // item takes about 0.75 of a tile's time, not 0.5: 24 KB of operands per 256 cycles of MMAs is
  // what an SM can pull).  Not with less than one whole round: 4 to 32 tiles measured 3-4 % slower
  // in halves.
  const uint32_t max_pairs = (uint32_t)a.sm_count / 2;
  const uint32_t rest = tiles % max_pairs;
  const bool split = !WIDE && a.force_bn == 0 && tiles > max_pairs && rest != 0 && 2 * rest <= max_pairs;  // a pinned width: whole tiles
  const uint32_t split_from = split ? tiles - rest : tiles;
  const uint32_t items = split_from + 2 * (tiles - split_from);
  const uint32_t pairs = items < max_pairs ? items : max_pairs;
  // bytes both CTAs report to the leader's stage barrier (operand copies count packed bytes)
  const uint32_t rows_per_cta = 128u + cfg::kBRows;
  const uint32_t op_bytes = (F4 || DENSE) ? rows_per_cta * 128u
                               : (uint32_t)(128 * BK * fmt_bits(a.fmtA) / 8 + cfg::kBRows * BK * fmt_bits(a.fmtB) / 8);
  const uint32_t tx_pair = 2u * op_bytes;  // the scale chunks complete on a barrier of their own
  const uint32_t op_bytes_half = (F4 || DENSE) ? (128u + 64u) * 128u
                                    : (uint32_t)(128 * BK * fmt_bits(a.fmtA) / 8 + 64 * BK * fmt_bits(a.fmtB) / 8);
  const uint32_t tx_half = 2u * op_bytes_half;
  // formats: kind::mxf4 encodes E2M1 as 1; kind::mxf8f6f4 uses the codes of mma_fmt_code();
  // kind::f16: BF16 = 1 for both operands, FP32 accumulator = 1 in bits [4,6), no scale-format bit.
  // N field = 256: the first (or only) MMA of a K step; the kernel derives the N = 128 one.
  const uint32_t fa = (F4 || DENSE) ? 1u : mma_fmt_code(a.fmtA), fb = (F4 || DENSE) ? 1u : mma_fmt_code(a.fmtB);
  const uint32_t idesc = (fa << 7) | (fb << 10) | (DENSE ? (1u << 4) : (1u << 23)) |
                         ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
  return launch_pdl(mx_gemm_pair_kernel<KIND, BN>, dim3(2 * pairs), dim3(kThreads), cfg::kSmemBytes, a.stream,
                    ma, mb, mb2, msa, msb, mc, (uint32_t)a.M, (uint32_t)a.N, (uint32_t)a.K, idesc, 8u, tx_pair,
                    epi_args(a), (uint32_t)a.batch, wait_budget(a), drop_fill(a), split_from, tx_half);
}

// M <= 128: operands swapped (see mx_gemm_skinny_kernel).
cudaError_t launch_skinny(const GemmArgs& a, EncodeTiledFn fn) {
  const uint32_t MP = ((uint32_t)a.M + 15u) / 16u * 16u;
  CUtensorMap mw, mx_, msw, msx;
  if (!make_operand_map(fn, &mw, a.B, a.fmtB, (uint64_t)a.N, (uint64_t)a.K, 128) ||
      !make_operand_map(fn, &mx_, a.A, a.fmtA, (uint64_t)a.M, (uint64_t)a.K, MP) ||
      !make_scale_map(fn, &msw, a.sB, (uint64_t)a.N, (uint64_t)a.K, 1) ||
      !make_scale_map(fn, &msx, a.sA, (uint64_t)a.M, (uint64_t)a.K, 1))
    return cudaErrorInvalidValue;
  // One CTA per SM: two K chunks per stage (with one, the per-stage hand-shakes -- about 550 cycles
  // for four small MMAs -- set the pace: 16 x 28672 x 8192 took 48.6 us with E4M3 weights and 41.5 us
  // with E2M1 weights, whose chunk is half the HBM bytes; with two 42.3 and 29.8 us; three or four,
  // i.e. fewer stages, are slower).  Where the tiles would need a second, partly empty round -- more
  // tiles than SMs, at most twice as many -- two CTAs share an SM instead (MP <= 96: half the shared
  // and tensor memory each, one chunk per stage): every tile is resident at once and an SM has two
  // MMA issuers (E2M1 weights 29.8 -> 27.2 us, 96 rows of E4M3 52.9 -> 50.9; slower outside that range).
  const uint32_t tiles = (uint32_t)((a.N + 127) / 128);
  const bool two = MP <= 96 && tiles > (uint32_t)a.sm_count && tiles <= 2u * (uint32_t)a.sm_count;
  const uint32_t kch = two ? 1u : 2u;
  const uint32_t budget = kch == 1 ? 232448u / 2 : 232448u;
  const uint32_t stage_bytes = kch * (16384u + MP * 128u + 1024u);
  const uint32_t fixed = kSkinnyBars * 8u + 16u + 1024u;  // barriers, TMEM slot + abort flag, alignment slack
  uint32_t stages = (budget - fixed) / stage_bytes;
  if (stages > kSkinnyMaxStages / kch) stages = kSkinnyMaxStages / kch;
  if (kch == 1 && stages > 8) stages = 8;  // 8 scale columns per stage behind column 192 of 256
  const SkinnyTmem tm = kch == 1 ? SkinnyTmem{256u, 96u, 192u} : SkinnyTmem{(uint32_t)kTmemCols, 128u, 256u};
  const uint32_t smem = stages * stage_bytes + fixed;
  static bool attr_set[64] = {false};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    e = cudaFuncSetAttribute(mx_gemm_skinny_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  const uint32_t slots = (kch == 1 ? 2u : 1u) * (uint32_t)a.sm_count;
  const uint32_t grid = tiles < slots ? tiles : slots;
  // bytes the two operand copies report (packed source bytes, rows past the end included)
  const uint32_t tx_bytes = (uint32_t)(128 * BK * fmt_bits(a.fmtB) / 8) + MP * (uint32_t)(BK * fmt_bits(a.fmtA) / 8);
  // the MMA's A side is B (format field [7,10)), its B side is A ([10,13)); N field = MP, M = 128
  const uint32_t idesc = (mma_fmt_code(a.fmtB) << 7) | (mma_fmt_code(a.fmtA) << 10) | (1u << 23) |
                         ((MP >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
  return launch_pdl(mx_gemm_skinny_kernel, dim3(grid), dim3(kThreads), smem, a.stream, mw, mx_, msw, msx, a.C,
                    (uint32_t)a.M, (uint32_t)a.N, (uint32_t)a.K, MP, idesc, tx_bytes, stages, kch, a.c_bf16 ? 1u : 0u,
                    wait_budget(a), drop_fill(a), tm);
}

}  // namespace

int launch_gemm(const GemmArgs& a, cudaError_t* cuda_err) {
  *cuda_err = cudaSuccess;
  EncodeTiledFn fn = encode_fn(cuda_err);
  if (!fn) return MX_ERR_CUDA;
  // few rows of A: operands swapped, deep ring (see mx_gemm_skinny_kernel)
  if (!a.dense && a.batch == 1 && a.q_elems == nullptr && a.M <= a.skinny_m) {
    *cuda_err = launch_skinny(a, fn);
    return *cuda_err == cudaSuccess ? MX_OK : MX_ERR_CUDA;
  }
  // One-CTA kernel: 256-wide tiles move the fewest operand bytes through shared memory per flop;
  // problems with fewer such tiles than SMs use 128-wide tiles to occupy more SMs.
  const int64_t tiles256 = a.batch * ((a.M + BM - 1) / BM) * ((a.N + 255) / 256);
  const int bn = tiles256 >= a.sm_count ? 256 : 128;
  // Two-CTA kernel or one-CTA kernel: by waves x time per tile.  Measured on tiles with K = 4096, in
  // units of a pair's 256 x 256 tile: a 128 x 256 tile of the one-CTA kernel takes 1.05 (8320 x 8192:
  // 14.6 us a wave against 13.9), a 128 x 128 tile 0.82 (512 x 4096 x 4096, 32 pair tiles or 128 single
  // ones: 0.73 against 0.88 PFLOP/s; 768 x 4096, 48 or 192: 1.09 against 0.87) -- both are bound by
  // operand delivery, of which the pair needs half per flop.  The pair kernel's tiles may be ragged in
  // M as in N (rows past M are zero-filled on the way in and clipped on the way out), except for
  // stacked matrices and the quantizing epilogue, which need whole tiles.
  const int64_t tiles_pair = a.batch * ((a.M + 255) / 256) * ((a.N + 255) / 256);
  const int64_t tiles_one = a.batch * ((a.M + BM - 1) / BM) * ((a.N + bn - 1) / bn);
  const int64_t pairs = a.sm_count / 2;
  // (a last round of at most half the pairs runs as half-width items, see launch_pair: about 0.75)
  const int64_t rest_pair = tiles_pair % pairs;
  const double cost_pair = (a.force_bn == 0 && tiles_pair > pairs && rest_pair != 0 && 2 * rest_pair <= pairs)
                               ? (double)(tiles_pair / pairs) + 0.75
                               : (double)((tiles_pair + pairs - 1) / pairs);
  const double cost_one = (double)((tiles_one + a.sm_count - 1) / a.sm_count) * (bn == 256 ? 1.05 : 0.82);
  const bool pair_ok = a.M % 256 == 0 || (a.batch == 1 && a.q_elems == nullptr);
  if (pair_ok && a.M >= 256 && cost_pair < cost_one) {
    // FP4 x FP4 with whole 256-element K stages runs on kind::mxf4 (twice the MMA rate)
    const bool f4 = !a.dense && a.fmtA == MX_E2M1 && a.fmtB == MX_E2M1 && a.K % 256 == 0;
    // 256 x 384 tiles pull fewer operand bytes per MAC from L2; taken only when pinned (force_bn):
    // a tie with 256 x 256 on the large configurations
    const int64_t tiles384 = a.batch * ((a.M + 255) / 256) * ((a.N + 383) / 384);
    const bool wide = a.q_elems == nullptr && a.force_bn == 384 && tiles384 >= a.sm_count / 2;
    if (wide)
      *cuda_err = a.dense ? launch_pair<2, 384>(a, fn) : f4 ? launch_pair<1, 384>(a, fn) : launch_pair<0, 384>(a, fn);
    else
      *cuda_err = a.dense ? launch_pair<2, 256>(a, fn) : f4 ? launch_pair<1, 256>(a, fn) : launch_pair<0, 256>(a, fn);
    return *cuda_err == cudaSuccess ? MX_OK : MX_ERR_CUDA;
  }
  CUtensorMap ma, mb;
  const bool ok =
      a.dense ? make_dense_map(fn, &ma, a.A, (uint64_t)(a.batch * a.M), (uint64_t)a.K, BM) &&
                    make_dense_map(fn, &mb, a.B, (uint64_t)(a.batch * a.N), (uint64_t)a.K, (uint32_t)bn)
              : make_operand_map(fn, &ma, a.A, a.fmtA, (uint64_t)(a.batch * a.M), (uint64_t)a.K, BM) &&
                    make_operand_map(fn, &mb, a.B, a.fmtB, (uint64_t)(a.batch * a.N), (uint64_t)a.K, (uint32_t)bn);
  if (!ok) {
    *cuda_err = cudaErrorInvalidValue;
    return MX_ERR_CUDA;
  }
  if (a.dense) {
    // kind::f16: FP32 accumulator (bits [4,6) = 1), BF16 operands (1), K-major A and B, M = 128
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BM >> 4) << 24);
    *cuda_err = bn == 256 ? launch_bn<256, true>(a, ma, mb, idesc) : launch_bn<128, true>(a, ma, mb, idesc);
  } else {
    // a_format [7,10), b_format [10,13), K-major A and B, scale format E8M0 (bit 23), M = 128
    const uint32_t idesc = (mma_fmt_code(a.fmtA) << 7) | (mma_fmt_code(a.fmtB) << 10) | (1u << 23) |
                           ((uint32_t)(BM >> 4) << 24);
    *cuda_err = bn == 256 ? launch_bn<256, false>(a, ma, mb, idesc) : launch_bn<128, false>(a, ma, mb, idesc);
  }
  return *cuda_err == cudaSuccess ? MX_OK : MX_ERR_CUDA;
}

// Implicit-GEMM convolution on the one-CTA kernel with 128 x 128 tiles (see mx_conv_kernel).
int launch_conv(const ConvArgs& a, cudaError_t* cuda_err) {
  *cuda_err = cudaSuccess;
  EncodeTiledFn fn = encode_fn(cuda_err);
  if (!fn) return MX_ERR_CUDA;
  constexpr int BN = 128;
  using cfg = Cfg<BN>;
  const int64_t M = a.N * a.Ho * a.Wo, K = (int64_t)a.kh * a.kw * a.C;
  GemmArgs ga = {};
  ga.C = a.y; ga.c_bf16 = a.y_bf16; ga.batch = 1; ga.M = M; ga.N = a.Cout; ga.K = K;
  CUtensorMap mb, msb, mc;
  if (!make_out_map(fn, &mc, ga) || !make_operand_map(fn, &mb, a.w_elems, a.fmt_w, (uint64_t)a.Cout, (uint64_t)K, BN) ||
      !make_scale_map(fn, &msb, a.w_scales, (uint64_t)a.Cout, (uint64_t)K, cfg::kSfbChunks)) {
    *cuda_err = cudaErrorInvalidValue;
    return MX_ERR_CUDA;
  }
  static bool attr_set[64] = {false};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess && (dev < 0 || dev >= 64 || !attr_set[dev])) {
    e = cudaFuncSetAttribute(mx_conv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cfg::kSmemBytes);
    if (e == cudaSuccess && dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  if (e != cudaSuccess) {
    *cuda_err = e;
    return MX_ERR_CUDA;
  }
  // im2col-mode map over x[N, H, W, C] (dims C, W, H, N): 128 channels x 128 pixels per copy, the
  // pixels walked along W, H, N with the convolution's strides inside the box of base positions
  // [-pad, extent + pad - (k - 1) dilation); usable when a 128-element K chunk lies in one tap
  CUtensorMap mx_ = mb;
  const bool tma = a.C % 128 == 0 && (a.kw - 1) * a.dil_w < 256 && (a.kh - 1) * a.dil_h < 256 && a.pad_w <= 127 &&
                   a.pad_h <= 127 && a.stride_w <= 8 && a.stride_h <= 8;
  if (tma) {
    Im2colFn im2col = im2col_fn(cuda_err);
    if (!im2col) return MX_ERR_CUDA;
    const cuuint64_t dims[4] = {(cuuint64_t)a.C, (cuuint64_t)a.W, (cuuint64_t)a.H, (cuuint64_t)a.N};
    const cuuint64_t strides[3] = {(cuuint64_t)a.C, (cuuint64_t)a.C * a.W, (cuuint64_t)a.C * a.W * a.H};
    const int lower[2] = {-a.pad_w, -a.pad_h};
    const int upper[2] = {a.pad_w - (a.kw - 1) * a.dil_w, a.pad_h - (a.kh - 1) * a.dil_h};
    const cuuint32_t estr[4] = {1, (cuuint32_t)a.stride_w, (cuuint32_t)a.stride_h, 1};
    if (im2col(&mx_, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<uint8_t*>(a.x_elems), dims, strides, lower, upper, 128,
               128, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
      *cuda_err = cudaErrorInvalidValue;
      return MX_ERR_CUDA;
    }
  }
  ConvGeom g;
  g.tma = tma ? 1u : 0u;
  g.x_codes = a.x_elems; g.x_scales = a.x_scales;
  g.H = (uint32_t)a.H; g.W = (uint32_t)a.W; g.Ho = (uint32_t)a.Ho; g.Wo = (uint32_t)a.Wo; g.kw = (uint32_t)a.kw;
  g.C = (uint32_t)a.C; g.cb = (uint32_t)(a.C / 32); g.kblocks = (uint32_t)(K / 32); g.M = (uint32_t)M;
  g.x_rows = (uint32_t)(a.N * a.H * a.W); g.x_layout = (uint32_t)a.x_layout;
  g.stride_h = a.stride_h; g.stride_w = a.stride_w; g.pad_h = a.pad_h; g.pad_w = a.pad_w;
  g.dil_h = a.dil_h; g.dil_w = a.dil_w;
  g.d_wo = make_fastdiv(g.Wo); g.d_howo = make_fastdiv(g.Ho * g.Wo); g.d_kw = make_fastdiv(g.kw);
  g.d_cb = make_fastdiv(g.cb);
  EpiArgs epi;
  epi.mode = a.y_bf16 ? 1u : 0u; epi.fmt = 0; epi.sticky = 0; epi.elems = nullptr; epi.scales = nullptr;
  const uint32_t tiles = (uint32_t)((M + BM - 1) / BM) * (uint32_t)((a.Cout + BN - 1) / BN);
  // 256 x 256 tiles on CTA pairs where the codes come through the im2col map and that costs fewer
  // waves (same weighting as launch_gemm: a 128 x 128 tile takes 0.82 of a pair tile's time)
  const int64_t tiles_pair = ((M + 255) / 256) * ((a.Cout + 255) / 256), pairs = a.sm_count / 2;
  const double cost_pair = (double)((tiles_pair + pairs - 1) / pairs);
  const double cost_one = (double)((tiles + a.sm_count - 1) / a.sm_count) * 0.82;
  if (tma && M >= 256 && cost_pair < cost_one) {
    using cfg2 = Cfg2<0, 256>;
    CUtensorMap msb2;
    if (!make_scale_map_k(fn, &msb2, a.w_scales, (uint64_t)a.Cout, (uint64_t)K, cfg2::kSfbGroups, cfg2::kKChunks)) {
      *cuda_err = cudaErrorInvalidValue;
      return MX_ERR_CUDA;
    }
    static bool attr2_set[64] = {false};
    if (dev < 0 || dev >= 64 || !attr2_set[dev]) {
      e = cudaFuncSetAttribute(mx_conv_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cfg2::kConvSmemBytes);
      if (e != cudaSuccess) {
        *cuda_err = e;
        return MX_ERR_CUDA;
      }
      if (dev >= 0 && dev < 64) attr2_set[dev] = true;
    }
    const uint32_t np = tiles_pair < pairs ? (uint32_t)tiles_pair : (uint32_t)pairs;
    // bytes both CTAs report to the leader's stage barrier: 128 x 128 codes of x and 128 rows of the filter each
    const uint32_t tx_pair = 2u * (uint32_t)(128 * BK + 128 * BK * fmt_bits(a.fmt_w) / 8);
    const uint32_t idesc2 = (mma_fmt_code(a.fmt_x) << 7) | (mma_fmt_code(a.fmt_w) << 10) | (1u << 23) |
                            ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
    *cuda_err = launch_pdl(mx_conv_pair_kernel, dim3(2 * np), dim3(kThreads), cfg2::kConvSmemBytes, a.stream, mx_, mb,
                              msb2, mc, (uint32_t)M, (uint32_t)a.Cout, (uint32_t)K, idesc2, 8u, tx_pair, epi, kSpinLimit, g);
    return *cuda_err == cudaSuccess ? MX_OK : MX_ERR_CUDA;
  }
  const uint32_t grid = tiles < (uint32_t)a.sm_count ? tiles : (uint32_t)a.sm_count;
  // the filter tile, plus the 128 x 128 codes of x when they come through the im2col map
  const uint32_t tx_bytes = (uint32_t)(BN * BK * fmt_bits(a.fmt_w) / 8) + (tma ? (uint32_t)(BM * BK) : 0u);
  const uint32_t idesc = (mma_fmt_code(a.fmt_x) << 7) | (mma_fmt_code(a.fmt_w) << 10) | (1u << 23) |
                         ((uint32_t)(BM >> 4) << 24) | ((uint32_t)(BN >> 3) << 17);
  *cuda_err = launch_pdl(mx_conv_kernel, dim3(grid), dim3(kConvThreads), cfg::kSmemBytes, a.stream, mx_, mb, msb,
                            mc, (uint32_t)M, (uint32_t)a.Cout, (uint32_t)K, idesc, 16u, tx_bytes, epi, kSpinLimit, g);
  return *cuda_err == cudaSuccess ? MX_OK : MX_ERR_CUDA;
}

// Reads and clears the device status word (synchronises the stream first).
int gemm_status(cudaStream_t stream, unsigned int* out, cudaError_t* cuda_err) {
  *cuda_err = cudaStreamSynchronize(stream);
  if (*cuda_err != cudaSuccess) return MX_ERR_CUDA;
  *cuda_err = cudaMemcpyFromSymbol(out, g_gemm_status, sizeof(unsigned int));
  if (*cuda_err != cudaSuccess) return MX_ERR_CUDA;
  if (*out != 0) {
    const unsigned int zero = 0;
    *cuda_err = cudaMemcpyToSymbol(g_gemm_status, &zero, sizeof(unsigned int));
    if (*cuda_err != cudaSuccess) return MX_ERR_CUDA;
  }
  return MX_OK;
}

}  // namespace mx

