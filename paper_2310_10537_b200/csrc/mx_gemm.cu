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
// Kernel structure (one CTA per SM, persistent over output tiles):
//   warp 0    TMA producer: packed A / B tiles (the sub-byte tensor-map types
//             expand FP6 / FP4 to one byte per element on the way in) and the
//             512-byte swizzled scale chunks -> shared-memory ring
//   warp 1    MMA issuer: scales shared -> tensor memory (tcgen05.cp), four
//             MMAs per stage, tcgen05.commit releases the stage / the accumulator
//   warps 2-5 epilogue: tensor memory -> registers -> FP32 C
// Every wait on an mbarrier is bounded; on expiry the kernel records a status
// word, raises a CTA-wide abort flag and every role falls through to the common
// exit, where tensor memory is released.
#include <cuda.h>  // CUtensorMap and enums only: the driver entry point is looked up at run time
#include <cuda_runtime.h>

#include <cstring>

#include "mx.h"
#include "mx_launch.h"

namespace mx {
namespace {

constexpr int BM = 128;         // rows of C per tile (= MMA M, one TMEM lane per row)
constexpr int BK = 128;         // K elements per pipeline stage: 4 MX blocks, 4 MMAs
constexpr int kMmaK = 32;       // K of one kind::mxf8f6f4 MMA = the MX block size
constexpr int kThreads = 192;   // 6 warps
constexpr int kTmemCols = 512;  // whole tensor memory of the SM (one CTA per SM)
constexpr long long kSpinLimit = 2000000000LL;  // cycles (~1 s) before a wait gives up

enum : unsigned int {
  ST_OK = 0,
  ST_PRODUCER_WAIT = 1,    // producer: stage never became empty
  ST_MMA_WAIT_FULL = 2,    // MMA issuer: stage never became full
  ST_MMA_WAIT_ACC = 3,     // MMA issuer: accumulator never drained
  ST_EPILOGUE_WAIT = 4,    // epilogue: accumulator never became full
};

// First failure of any GEMM launch on this device since the last check (0 = none).
__device__ unsigned int g_gemm_status;

template <int BN>
struct Cfg {
  static_assert(BN == 128 || BN == 192 || BN == 256, "tile width");
  static constexpr int kStages = BN == 256 ? 4 : (BN == 192 ? 5 : 6);
  static constexpr int kAccStages = BN == 256 ? 1 : 2;
  // 512-byte scale chunks (128 rows each) of B per stage; a 192-wide tile starts on a
  // 64-row boundary and always lies inside two consecutive chunks
  static constexpr int kSfbChunks = BN == 128 ? 1 : 2;
  static constexpr int kSfCols = 4 + 4 * kSfbChunks;       // TMEM columns of scales per stage
  static constexpr int kSfCol0 = kAccStages * BN;          // first scale column
  static constexpr uint32_t kABytes = BM * BK;             // one byte per element in shared memory
  static constexpr uint32_t kBBytes = BN * BK;
  static constexpr uint32_t kSfBytes = 512 * (1 + kSfbChunks);
  static constexpr uint32_t kOffA = 0;
  static constexpr uint32_t kOffB = kOffA + kStages * kABytes;
  static constexpr uint32_t kOffSf = kOffB + kStages * kBBytes;
  static constexpr uint32_t kOffBar = kOffSf + kStages * kSfBytes;
  // barriers: full[S], empty[S], acc_full[A], acc_empty[A]; then tmem slot + abort flag
  static constexpr uint32_t kNumBars = 2 * kStages + 2 * kAccStages;
  static constexpr uint32_t kSmemBytes = kOffBar + kNumBars * 8 + 16 + 1024;  // + alignment slack
  static_assert(kSfCol0 + kStages * kSfCols <= kTmemCols, "tensor memory budget");
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
// Bounded wait: false if the abort flag was raised or the cycle budget ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity,
                                          const volatile uint32_t* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 31u) == 0) {
      if (*abort_flag != 0) return false;
      if (clock64() - t0 > kSpinLimit) return false;
    }
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes,
                                          uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
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

struct TileCoord {
  uint32_t tm, tn;
};
// Output tiles are walked in bands of group_m tile rows so that the A band and
// the B tiles of a wave of CTAs stay in L2.
__device__ __forceinline__ TileCoord tile_coord(uint32_t t, uint32_t tiles_m, uint32_t tiles_n,
                                                uint32_t group_m) {
  const uint32_t per_group = group_m * tiles_n;
  const uint32_t g = t / per_group, r = t - g * per_group;
  const uint32_t first_m = g * group_m;
  const uint32_t gm = min(group_m, tiles_m - first_m);
  TileCoord c;
  c.tn = r / gm;
  c.tm = first_m + (r - c.tn * gm);
  return c;
}

__device__ __forceinline__ void raise_abort(volatile uint32_t* abort_flag, unsigned int code) {
  atomicCAS(&g_gemm_status, 0u, code);
  *abort_flag = 1u;
}

template <int BN>
__global__ void __launch_bounds__(kThreads, 1)
mx_gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
               const uint8_t* __restrict__ sA, const uint8_t* __restrict__ sB,
               float* __restrict__ C, uint32_t M, uint32_t N, uint32_t K, uint32_t idesc_base,
               uint32_t group_m, uint32_t c_aligned32, uint32_t tx_bytes) {
  using cfg = Cfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar0 = smem_base + cfg::kOffBar;
  auto full_bar = [&](uint32_t s) { return bar0 + 8 * s; };
  auto empty_bar = [&](uint32_t s) { return bar0 + 8 * (cfg::kStages + s); };
  auto acc_full_bar = [&](uint32_t a) { return bar0 + 8 * (2 * cfg::kStages + a); };
  auto acc_empty_bar = [&](uint32_t a) { return bar0 + 8 * (2 * cfg::kStages + cfg::kAccStages + a); };
  volatile uint32_t* tmem_slot =
      reinterpret_cast<volatile uint32_t*>(smem_gen + cfg::kOffBar + cfg::kNumBars * 8);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tiles_m = M / BM, tiles_n = (N + BN - 1) / BN, num_tiles = tiles_m * tiles_n;
  const uint32_t n_chunks128 = N / 128;  // scale chunks of B along N
  const uint32_t k_chunks = K / BK;

  if (threadIdx.x == 0) {
    for (uint32_t s = 0; s < cfg::kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (uint32_t a = 0; a < cfg::kAccStages; ++a) {
      mbar_init(acc_full_bar(a), 1);
      mbar_init(acc_empty_bar(a), 4);  // one arrival per epilogue warp
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_a)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_b)) : "memory");
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

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      for (uint32_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
        const TileCoord tc = tile_coord(t, tiles_m, tiles_n, group_m);
        for (uint32_t kc = 0; kc < k_chunks; ++kc) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) {
            raise_abort(abort_flag, ST_PRODUCER_WAIT);
            ok = false;
            break;
          }
          const uint32_t fb = full_bar(stage);
          // a ragged last tile (BN = 192) may reach past the last scale chunk of B
          const uint32_t sfb_first = tc.tn * BN / 128;
          const uint32_t sfb_have = min((uint32_t)cfg::kSfbChunks, n_chunks128 - sfb_first);
          mbar_arrive_expect_tx(fb, tx_bytes - 512u * (cfg::kSfbChunks - sfb_have));
          tma_load_2d(smem_base + cfg::kOffA + stage * cfg::kABytes, &tmap_a, (int)(kc * BK),
                      (int)(tc.tm * BM), fb);
          tma_load_2d(smem_base + cfg::kOffB + stage * cfg::kBBytes, &tmap_b, (int)(kc * BK),
                      (int)(tc.tn * BN), fb);
          const uint32_t sf = smem_base + cfg::kOffSf + stage * cfg::kSfBytes;
          bulk_load(sf, sA + ((size_t)tc.tm * k_chunks + kc) * 512, 512, fb);
#pragma unroll
          for (uint32_t j = 0; j < cfg::kSfbChunks; ++j)
            if (j < sfb_have)
              bulk_load(sf + 512 + 512 * j, sB + ((size_t)(sfb_first + j) * k_chunks + kc) * 512, 512, fb);
          if (++stage == cfg::kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {  // let copies that are still in flight land before the CTA goes away
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer -------------------------------
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
      bool ok = true;
      for (uint32_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
        if (!mbar_wait(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag)) {
          raise_abort(abort_flag, ST_MMA_WAIT_ACC);
          break;
        }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        // scales of row n of the tile sit in column (n0 % 128 + n) / 32 of the copied chunks
        const uint32_t sfb_col = 4 + ((tile_coord(t, tiles_m, tiles_n, group_m).tn * BN) % 128) / 32;
        for (uint32_t kc = 0; kc < k_chunks; ++kc) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag)) {
            raise_abort(abort_flag, ST_MMA_WAIT_FULL);
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t sf_smem = smem_base + cfg::kOffSf + stage * cfg::kSfBytes;
          const uint32_t sf_tmem = tmem_base + cfg::kSfCol0 + stage * cfg::kSfCols;
          tc_cp_scales(sf_tmem, scale_desc(sf_smem));
#pragma unroll
          for (uint32_t j = 0; j < cfg::kSfbChunks; ++j)
            tc_cp_scales(sf_tmem + 4 + 4 * j, scale_desc(sf_smem + 512 + 512 * j));
          const uint64_t adesc = operand_desc(smem_base + cfg::kOffA + stage * cfg::kABytes);
          const uint64_t bdesc = operand_desc(smem_base + cfg::kOffB + stage * cfg::kBBytes);
#pragma unroll
          for (uint32_t k = 0; k < BK / kMmaK; ++k) {
            // byte k of each 32-bit scale column belongs to MX block k of this stage
            const uint32_t idesc = idesc_base | (k << 4) | (k << 29);
            tc_mma(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, sf_tmem, sf_tmem + sfb_col,
                   (kc | k) != 0 ? 1u : 0u);
          }
          tc_commit(empty_bar(stage));  // the stage is free once these MMAs have read it
          if (++stage == cfg::kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) tc_commit(acc_full_bar(acc));
        if (++acc == cfg::kAccStages) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // -------------------------------- epilogue --------------------------------
    const uint32_t quarter = warp & 3u;  // TMEM lanes this warp may read: 32*quarter .. +31
    uint32_t acc = 0, acc_phase = 0;
    for (uint32_t t = blockIdx.x; t < num_tiles; t += gridDim.x) {
      const TileCoord tc = tile_coord(t, tiles_m, tiles_n, group_m);
      if (!mbar_wait(acc_full_bar(acc), acc_phase, abort_flag)) {
        if (lane == 0) raise_abort(abort_flag, ST_EPILOGUE_WAIT);
        break;
      }
      tc_fence_after();
      const uint32_t row = tc.tm * BM + quarter * 32 + lane;
      float* crow = C + (size_t)row * N + (size_t)tc.tn * BN;
      const uint32_t taddr = tmem_base + ((quarter * 32u) << 16) + acc * BN;
      const uint32_t valid_cols = min((uint32_t)BN, N - tc.tn * BN);  // multiple of 64
      // two register buffers: the load of chunk j+1 is in flight while chunk j is stored
      uint32_t r[2][32];
      tc_ld32(taddr, r[0]);
#pragma unroll
      for (uint32_t j = 0; j < BN / 32; ++j) {
        tc_wait_ld();
        if (j + 1 < BN / 32) tc_ld32(taddr + 32 * (j + 1), r[(j + 1) & 1]);
        const uint32_t c0 = 32 * j;
        if (c0 < valid_cols) {
          if (c_aligned32) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
              asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(crow + c0 + 8 * i),
                           "r"(r[j & 1][8 * i]), "r"(r[j & 1][8 * i + 1]), "r"(r[j & 1][8 * i + 2]),
                           "r"(r[j & 1][8 * i + 3]), "r"(r[j & 1][8 * i + 4]), "r"(r[j & 1][8 * i + 5]),
                           "r"(r[j & 1][8 * i + 6]), "r"(r[j & 1][8 * i + 7]) : "memory");
          } else {
#pragma unroll
            for (int i = 0; i < 8; ++i)
              *reinterpret_cast<uint4*>(crow + c0 + 4 * i) =
                  make_uint4(r[j & 1][4 * i], r[j & 1][4 * i + 1], r[j & 1][4 * i + 2], r[j & 1][4 * i + 3]);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty_bar(acc));
      if (++acc == cfg::kAccStages) { acc = 0; acc_phase ^= 1u; }
    }
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

// ---- host side ---------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn(cudaError_t* err) {
  static EncodeTiledFn fn = nullptr;
  if (fn) { *err = cudaSuccess; return fn; }
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q;
  *err = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
  if (*err != cudaSuccess) return nullptr;
  if (q != cudaDriverEntryPointSuccess || !p) { *err = cudaErrorNotSupported; return nullptr; }
  fn = (EncodeTiledFn)p;
  return fn;
}

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
  const cuuint64_t dims[2] = {K, rows};
  const cuuint64_t strides[1] = {K * (uint64_t)bits / 8};
  const cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, dt, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN>
cudaError_t launch_bn(const GemmArgs& a, const CUtensorMap& ma, const CUtensorMap& mb,
                      uint32_t idesc_base) {
  using cfg = Cfg<BN>;
  static bool attr_set[64] = {false};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    e = cudaFuncSetAttribute(mx_gemm_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)cfg::kSmemBytes);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  const uint32_t tiles = (uint32_t)(a.M / BM) * (uint32_t)((a.N + BN - 1) / BN);
  const uint32_t grid = tiles < (uint32_t)a.sm_count ? tiles : (uint32_t)a.sm_count;
  const uint32_t group_m = 16;
  // Bytes the producer's copies report to a stage's mbarrier: the tensor-map copies count the
  // packed source bytes (bits/8 per element), not the expanded shared-memory footprint.
  const uint32_t tx_bytes = (uint32_t)(BM * BK * fmt_bits(a.fmtA) / 8 + BN * BK * fmt_bits(a.fmtB) / 8) +
                            cfg::kSfBytes;
  mx_gemm_kernel<BN><<<grid, kThreads, cfg::kSmemBytes, a.stream>>>(
      ma, mb, a.sA, a.sB, a.C, (uint32_t)a.M, (uint32_t)a.N, (uint32_t)a.K,
      idesc_base | ((uint32_t)(BN >> 3) << 17), group_m, (uint32_t)((uintptr_t)a.C % 32 == 0),
      tx_bytes);
  return cudaGetLastError();
}

}  // namespace

int launch_gemm(const GemmArgs& a, cudaError_t* cuda_err) {
  *cuda_err = cudaSuccess;
  EncodeTiledFn fn = encode_fn(cuda_err);
  if (!fn) return MX_ERR_CUDA;
#ifdef MX_GEMM_BN
  const int bn = MX_GEMM_BN;
#else
  // 256-wide tiles move the fewest operand bytes through shared memory per flop; problems with
  // fewer such tiles than SMs use 128-wide tiles to occupy more SMs.
  const int64_t tiles256 = (a.M / BM) * ((a.N + 255) / 256);
  const int bn = tiles256 >= a.sm_count ? 256 : 128;
#endif
  CUtensorMap ma, mb;
  if (!make_operand_map(fn, &ma, a.A, a.fmtA, (uint64_t)a.M, (uint64_t)a.K, BM) ||
      !make_operand_map(fn, &mb, a.B, a.fmtB, (uint64_t)a.N, (uint64_t)a.K, (uint32_t)bn)) {
    *cuda_err = cudaErrorInvalidValue;
    return MX_ERR_CUDA;
  }
  // a_format [7,10), b_format [10,13), K-major A and B, scale format E8M0 (bit 23), M = 128
  const uint32_t idesc = (mma_fmt_code(a.fmtA) << 7) | (mma_fmt_code(a.fmtB) << 10) | (1u << 23) |
                         ((uint32_t)(BM >> 4) << 24);
  *cuda_err = bn == 256 ? launch_bn<256>(a, ma, mb, idesc)
              : bn == 192 ? launch_bn<192>(a, ma, mb, idesc) : launch_bn<128>(a, ma, mb, idesc);
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
