/*
 * mx_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow CPU restatement of what the MX paper (arXiv 2310.10537)
 * defines, used only to check the CUDA library and as the timed CPU baseline:
 *
 *   oracle_quantize    Section 3, Algorithm 1, one step after the other, in
 *                      integer and double arithmetic (every quantity on the
 *                      way is exactly representable in a double)
 *   oracle_dequantize  Section 2: v_i = X * P_i, NaN if X is NaN
 *   oracle_gemm        Section 4.1: the dot product of the dequantized
 *                      operands, written as its FP64 definition
 *
 * It shares no source, header, table or helper with the CUDA library (the enum
 * values below are restated, not included) and is loaded through ctypes by the
 * tests.  The only parallelism is an OpenMP "parallel for" over output rows.
 *
 * Readings taken where the paper is silent (listed with reasons in the design
 * notes of the repository):
 *   - all-zero block: scale byte 0x00, all elements zero, sign kept
 *   - shared_exp below -127: clamped to -127
 *   - block containing Inf or NaN: scale byte 0xFF (X = NaN), codes 0
 *   - results rounding to zero keep the sign bit (FP formats); INT8 gives 0
 *   - FP32-subnormal inputs are flushed before the maximum is taken
 *   - round first, then saturate to the largest normal
 *   - INT8: emax_elem = 0, value n/64, symmetric saturation at +-127
 *   - |X * P| above the FP32 range dequantizes to +-Inf
 *   - codes are a little-endian bit stream along the row
 *   - an axis whose length is not a multiple of 32 ends in a partial block: the
 *     elements that are missing are taken as +0 (they cannot change the block
 *     maximum and encode as code 0), and the stored row is padded with those
 *     zero codes to a whole block
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Same numeric values as the library's public enums (restated on purpose). */
enum { F_E4M3 = 0, F_E5M2 = 1, F_E3M2 = 2, F_E2M3 = 3, F_E2M1 = 4, F_INT8 = 5 };
enum { R_RNE = 0, R_RHAZ = 1 };
enum { T_F32 = 0, T_BF16 = 1, T_F64 = 2 };
enum { L_LINEAR = 0, L_SWIZZLED = 1 };

#define BLOCK 32

/* Table 1 names the formats; their parameters are those of the OCP FP8 and OCP
 * MX specifications the paper refers to in Section 2 ("Concrete MX Formats"). */
typedef struct {
  int bits;          /* width of a code                                */
  int ebits, mbits;  /* exponent and mantissa field widths             */
  int bias;          /* exponent bias                                  */
  int emax;          /* exponent of the largest normal ("emax_elem")   */
  double max_normal; /* largest normal magnitude                       */
} fmt_info;

static const fmt_info FMT[6] = {
    /* E4M3 */ {8, 4, 3, 7, 8, 448.0},
    /* E5M2 */ {8, 5, 2, 15, 15, 57344.0},
    /* E3M2 */ {6, 3, 2, 3, 4, 28.0},
    /* E2M3 */ {6, 2, 3, 1, 2, 7.5},
    /* E2M1 */ {4, 2, 1, 1, 2, 6.0},
    /* INT8 */ {8, 0, 6, 0, 0, 127.0 / 64.0},
};

static int fmt_ok(int fmt) { return fmt >= 0 && fmt <= 5; }

int oracle_fmt_bits(int fmt) { return fmt_ok(fmt) ? FMT[fmt].bits : 0; }
int oracle_fmt_emax(int fmt) { return fmt_ok(fmt) ? FMT[fmt].emax : -1; }
double oracle_fmt_max_normal(int fmt) { return fmt_ok(fmt) ? FMT[fmt].max_normal : 0.0; }

int oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ---------------------------------------------------------------------- */
/* Scalar helpers                                                          */
/* ---------------------------------------------------------------------- */

static uint32_t f32_bits(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }
static float bits_f32(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }

/* Read element idx of a float tensor as FP32 bits; BF16 widens exactly. */
static uint32_t load_bits(const void* in, int dtype, int64_t idx) {
  if (dtype == T_BF16) return (uint32_t)((const uint16_t*)in)[idx] << 16;
  return ((const uint32_t*)in)[idx];
}

/* round a non-negative exact quotient t to an integer */
static double round_mode(double t, int rounding) {
  double n = floor(t);
  double frac = t - n; /* exact: t has few significant bits */
  if (rounding == R_RHAZ) {
    if (frac >= 0.5) n += 1.0; /* ties away from zero (magnitude grows) */
  } else {
    if (frac > 0.5) n += 1.0;
    else if (frac == 0.5 && fmod(n, 2.0) == 1.0) n += 1.0; /* ties to even */
  }
  return n;
}

/*
 * The element cast of Section 3, Algorithm 1: the exact quotient r = V_i / X is
 * rounded onto the element format's grid and saturated at its largest normal
 * value.  sign is the sign bit of V_i.
 */
static uint8_t encode_element(double r, int sign, int fmt, int rounding) {
  const fmt_info* f = &FMT[fmt];
  double a = fabs(r);
  if (fmt == F_INT8) {
    double n = round_mode(a * 64.0, rounding);
    if (n > 127.0) n = 127.0;
    int v = (int)n;
    if (sign) v = -v;
    return (uint8_t)(v & 0xFF); /* two's complement; -0 is 0 */
  }
  int m = f->mbits;
  int emin = 1 - f->bias;
  uint32_t mag = 0;
  if (a != 0.0) {
    int ex;
    (void)frexp(a, &ex); /* a = frac * 2^ex, frac in [0.5, 1) */
    int e = ex - 1;      /* floor(log2 a) */
    if (e < emin) e = emin;
    double q = ldexp(1.0, e - m);          /* grid spacing in this binade */
    double n = round_mode(a / q, rounding); /* a / q is exact */
    double ap = n * q;
    if (ap > f->max_normal) ap = f->max_normal; /* saturate, sign kept */
    if (ap == 0.0) {
      mag = 0;
    } else if (ap < ldexp(1.0, emin)) { /* subnormal of the element format */
      mag = (uint32_t)(ap / ldexp(1.0, emin - m));
    } else {
      int ex2;
      (void)frexp(ap, &ex2);
      int e2 = ex2 - 1;
      uint32_t expfield = (uint32_t)(e2 + f->bias);
      uint32_t mant = (uint32_t)(ap / ldexp(1.0, e2 - m)) - (1u << m);
      mag = (expfield << m) | mant;
    }
  }
  return (uint8_t)(((uint32_t)(sign ? 1 : 0) << (f->ebits + m)) | mag);
}

/* Value of one element code (Section 2.1 for the special codes). */
static double decode_element(uint8_t code, int fmt) {
  const fmt_info* f = &FMT[fmt];
  if (fmt == F_INT8) return (double)(int8_t)code / 64.0;
  int m = f->mbits, eb = f->ebits;
  uint32_t c = code & ((1u << f->bits) - 1u);
  int sign = (c >> (eb + m)) & 1;
  uint32_t expfield = (c >> m) & ((1u << eb) - 1u);
  uint32_t mant = c & ((1u << m) - 1u);
  double v;
  if (fmt == F_E4M3 && expfield == 15 && mant == 7) return NAN;
  if (fmt == F_E5M2 && expfield == 31) {
    if (mant == 0) return sign ? -INFINITY : INFINITY;
    return NAN;
  }
  if (expfield == 0) v = ldexp((double)mant, 1 - f->bias - m);
  else v = ldexp((double)((1u << m) | mant), (int)expfield - f->bias - m);
  return sign ? -v : v;
}

uint8_t oracle_encode_element(double r, int fmt, int rounding) {
  if (!fmt_ok(fmt)) return 0;
  return encode_element(r, signbit(r) ? 1 : 0, fmt, rounding);
}
double oracle_decode_element(uint8_t code, int fmt) {
  if (!fmt_ok(fmt)) return NAN;
  return decode_element(code, fmt);
}

/* ---------------------------------------------------------------------- */
/* Layout helpers                                                          */
/* ---------------------------------------------------------------------- */

size_t oracle_scales_bytes(int64_t rows, int64_t kblocks, int layout) {
  if (layout == L_LINEAR) return (size_t)(rows * kblocks);
  return (size_t)(((rows + 127) / 128) * ((kblocks + 3) / 4) * 512);
}

size_t oracle_scale_offset(int64_t row, int64_t kb, int64_t rows, int64_t kblocks, int layout) {
  (void)rows;
  if (layout == L_LINEAR) return (size_t)(row * kblocks + kb);
  int64_t kchunks = (kblocks + 3) / 4;
  int64_t chunk = (row / 128) * kchunks + kb / 4;
  return (size_t)(chunk * 512 + (row % 32) * 16 + ((row % 128) / 32) * 4 + kb % 4);
}

size_t oracle_elems_bytes(int64_t rows, int64_t L, int fmt) {
  return (size_t)(rows * L * FMT[fmt].bits / 8);
}

/* code i of a row occupies bits [w*i, w*i+w) of a little-endian bit stream */
static void put_code(uint8_t* row, int64_t i, int w, uint8_t code) {
  for (int b = 0; b < w; ++b) {
    int64_t bit = i * w + b;
    if ((code >> b) & 1) row[bit >> 3] |= (uint8_t)(1u << (bit & 7));
  }
}
static uint8_t get_code(const uint8_t* row, int64_t i, int w) {
  uint8_t code = 0;
  for (int b = 0; b < w; ++b) {
    int64_t bit = i * w + b;
    if ((row[bit >> 3] >> (bit & 7)) & 1) code |= (uint8_t)(1u << b);
  }
  return code;
}

void oracle_pack_codes(const uint8_t* codes, int64_t n, int fmt, uint8_t* out) {
  int w = FMT[fmt].bits;
  memset(out, 0, (size_t)(n * w / 8));
  for (int64_t i = 0; i < n; ++i) put_code(out, i, w, codes[i]);
}
void oracle_unpack_codes(const uint8_t* packed, int64_t n, int fmt, uint8_t* codes) {
  int w = FMT[fmt].bits;
  for (int64_t i = 0; i < n; ++i) codes[i] = get_code(packed, i, w);
}

/* ---------------------------------------------------------------------- */
/* Algorithm 1 on one block                                                */
/* ---------------------------------------------------------------------- */

/* Section 3, Algorithm 1.  bits[32]: FP32 bit patterns of V_1..V_32.  The shared exponent is
 * the exponent of the block maximum less the element format's largest exponent; the scale is
 * that power of two; every element is divided by it and cast with saturation.  Writes 32 codes
 * and the scale byte. */
static void quantize_block_bits(const uint32_t* bits, int fmt, int rounding,
                                uint8_t* codes, uint8_t* scale_byte) {
  uint32_t v[BLOCK];
  int nonfinite = 0;
  uint32_t amax_bits = 0; /* magnitude bits: ordering of positive floats = ordering of bits */
  for (int i = 0; i < BLOCK; ++i) {
    uint32_t u = bits[i];
    uint32_t expfield = (u >> 23) & 0xFF;
    if (expfield == 0) u &= 0x80000000u; /* FP32 subnormal (or zero) -> signed zero */
    if (expfield == 0xFF) nonfinite = 1; /* Inf or NaN */
    v[i] = u;
    uint32_t mag = u & 0x7FFFFFFFu;
    if (mag > amax_bits) amax_bits = mag;
  }
  if (nonfinite) { /* X = NaN makes the whole block NaN (Section 2) */
    *scale_byte = 0xFF;
    memset(codes, 0, BLOCK);
    return;
  }
  int shared_exp;
  if (amax_bits == 0) {
    shared_exp = -127; /* log2(0): smallest scale */
  } else {
    int E = (int)((amax_bits >> 23) & 0xFF) - 127; /* floor(log2(amax)), amax is normal */
    shared_exp = E - FMT[fmt].emax;                /* shared exponent */
    if (shared_exp < -127) shared_exp = -127;
    if (shared_exp > 127) shared_exp = 127;
  }
  *scale_byte = (uint8_t)(shared_exp + 127); /* X = 2^shared_exp as an E8M0 byte */
  for (int i = 0; i < BLOCK; ++i) {           /* the elements, each scaled by 1/X and cast */
    double V = (double)bits_f32(v[i]);
    double r = ldexp(V, -shared_exp); /* V / X, exact in double */
    codes[i] = encode_element(r, (int)(v[i] >> 31), fmt, rounding);
  }
}

int oracle_quantize_block(const float* v32, int fmt, int rounding, uint8_t* codes32,
                          uint8_t* scale_byte) {
  if (!fmt_ok(fmt)) return -3;
  uint32_t bits[BLOCK];
  for (int i = 0; i < BLOCK; ++i) bits[i] = f32_bits(v32[i]);
  quantize_block_bits(bits, fmt, rounding, codes32, scale_byte);
  return 0;
}

/* ---------------------------------------------------------------------- */
/* Whole tensors                                                           */
/* ---------------------------------------------------------------------- */

/*
 * in: contiguous [outer, L, inner]; blocks run along L (the principal axis of
 * Section 3's last paragraph).  Output row o*inner + j holds the blocks of
 * in[o, :, j] in order, so the shared-scale axis is innermost in the output.
 */
int oracle_quantize(const void* in, int in_dtype, int64_t outer, int64_t L, int64_t inner,
                    int fmt, int rounding, int scale_layout, uint8_t* elems, uint8_t* scales) {
  if (!fmt_ok(fmt)) return -3;
  if (L < 0 || outer < 0 || inner < 0) return -2;
  const int w = FMT[fmt].bits;
  const int64_t rows = outer * inner, kblocks = (L + BLOCK - 1) / BLOCK;
  const int64_t row_bytes = kblocks * BLOCK * w / 8; /* rows padded to whole blocks */
  memset(elems, 0, (size_t)(rows * row_bytes));
  memset(scales, 0, oracle_scales_bytes(rows, kblocks, scale_layout)); /* padding = 0x00 */
#pragma omp parallel for schedule(static)
  for (int64_t row = 0; row < rows; ++row) {
    const int64_t o = row / inner, j = row % inner;
    uint8_t* out_row = elems + row * row_bytes;
    for (int64_t b = 0; b < kblocks; ++b) {
      uint32_t bits[BLOCK];
      uint8_t codes[BLOCK], sb;
      for (int i = 0; i < BLOCK; ++i) /* positions past the end of the axis: +0 */
        bits[i] = b * BLOCK + i < L ? load_bits(in, in_dtype, (o * L + (b * BLOCK + i)) * inner + j) : 0u;
      quantize_block_bits(bits, fmt, rounding, codes, &sb);
      for (int i = 0; i < BLOCK; ++i) put_code(out_row, b * BLOCK + i, w, codes[i]);
      scales[oracle_scale_offset(row, b, rows, kblocks, scale_layout)] = sb;
    }
  }
  return 0;
}

/* v = X * P in double (always exact), or NaN when X is NaN. */
static double dequant_value(uint8_t code, uint8_t scale_byte, int fmt) {
  if (scale_byte == 0xFF) return NAN;
  double p = decode_element(code, fmt);
  return ldexp(p, (int)scale_byte - 127);
}

static float to_f32(double v) {
  if (isnan(v)) return bits_f32(0x7FC00000u);
  if (fabs(v) > 3.4028234663852886e38) return v < 0 ? -INFINITY : INFINITY;
  return (float)v; /* exact: <= 7 significant bits, least bit >= 2^-143 */
}

static uint16_t to_bf16(double v) {
  if (isnan(v)) return 0x7FC0;
  float f = to_f32(v);
  uint32_t u = f32_bits(f);
  if ((u & 0x7F800000u) == 0x7F800000u) return (uint16_t)(u >> 16); /* Inf */
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb; /* round to nearest, ties to even, on the low 16 bits */
  return (uint16_t)(u >> 16);
}

int oracle_dequantize(const uint8_t* elems, const uint8_t* scales, int64_t rows, int64_t L,
                      int fmt, int scale_layout, int out_dtype, void* out) {
  if (!fmt_ok(fmt)) return -3;
  if (L < 0) return -2;
  const int w = FMT[fmt].bits;
  const int64_t kblocks = (L + BLOCK - 1) / BLOCK, row_bytes = kblocks * BLOCK * w / 8;
#pragma omp parallel for schedule(static)
  for (int64_t row = 0; row < rows; ++row) {
    const uint8_t* in_row = elems + row * row_bytes;
    for (int64_t k = 0; k < L; ++k) {
      uint8_t sb = scales[oracle_scale_offset(row, k / BLOCK, rows, kblocks, scale_layout)];
      double v = dequant_value(get_code(in_row, k, w), sb, fmt);
      int64_t idx = row * L + k;
      if (out_dtype == T_F64) ((double*)out)[idx] = v;
      else if (out_dtype == T_BF16) ((uint16_t*)out)[idx] = to_bf16(v);
      else ((float*)out)[idx] = to_f32(v);
    }
  }
  return 0;
}

/*
 * C64[m,n] = sum_k a[m,k] * b[n,k],  S[m,n] = sum_k |a[m,k]| * |b[n,k]|
 * with a, b the dequantized operands in double.  A is [M x K], B is [N x K],
 * both with the shared-scale axis (K) innermost.  Either output may be NULL.
 */
int oracle_gemm(const uint8_t* A, const uint8_t* sA, const uint8_t* B, const uint8_t* sB,
                int64_t M, int64_t N, int64_t K, int fmtA, int fmtB, int scale_layout,
                double* C64, double* S) {
  if (!fmt_ok(fmtA) || !fmt_ok(fmtB)) return -3;
  if (K % BLOCK != 0) return -2;
  double* a = (double*)malloc((size_t)(M * K) * sizeof(double));
  double* b = (double*)malloc((size_t)(N * K) * sizeof(double));
  if (!a || !b) { free(a); free(b); return -9; }
  oracle_dequantize(A, sA, M, K, fmtA, scale_layout, T_F64, a);
  oracle_dequantize(B, sB, N, K, fmtB, scale_layout, T_F64, b);
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m) {
    for (int64_t n = 0; n < N; ++n) {
      double acc = 0.0, sabs = 0.0;
      for (int64_t k = 0; k < K; ++k) {
        double p = a[m * K + k] * b[n * K + k];
        acc += p;
        sabs += fabs(p);
      }
      if (C64) C64[m * N + n] = acc;
      if (S) S[m * N + n] = sabs;
    }
  }
  free(a);
  free(b);
  return 0;
}

/* The same sums for a list of (m, n) positions, operands read straight from
 * the packed tensors: used on problems too large for the full triple loop. */
int oracle_gemm_samples(const uint8_t* A, const uint8_t* sA, const uint8_t* B, const uint8_t* sB,
                        int64_t M, int64_t N, int64_t K, int fmtA, int fmtB, int scale_layout,
                        const int64_t* ms, const int64_t* ns, int64_t count,
                        double* c_out, double* s_out) {
  if (!fmt_ok(fmtA) || !fmt_ok(fmtB)) return -3;
  if (K % BLOCK != 0) return -2;
  const int wa = FMT[fmtA].bits, wb = FMT[fmtB].bits;
  const int64_t kblocks = K / BLOCK;
#pragma omp parallel for schedule(dynamic, 16)
  for (int64_t s = 0; s < count; ++s) {
    const int64_t m = ms[s], n = ns[s];
    const uint8_t* arow = A + m * (K * wa / 8);
    const uint8_t* brow = B + n * (K * wb / 8);
    double acc = 0.0, sabs = 0.0;
    for (int64_t k = 0; k < K; ++k) {
      uint8_t sa = sA[oracle_scale_offset(m, k / BLOCK, M, kblocks, scale_layout)];
      uint8_t sb = sB[oracle_scale_offset(n, k / BLOCK, N, kblocks, scale_layout)];
      double p = dequant_value(get_code(arow, k, wa), sa, fmtA) *
                 dequant_value(get_code(brow, k, wb), sb, fmtB);
      acc += p;
      sabs += fabs(p);
    }
    c_out[s] = acc;
    s_out[s] = sabs;
  }
  return 0;
}
