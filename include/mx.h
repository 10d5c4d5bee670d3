/*
 * mx.h -- C ABI of the Microscaling (MX) hot path for NVIDIA B200 (sm_100a).
 *
 * The library implements, as hand-written CUDA kernels, the three operations
 * the MX paper (arXiv 2310.10537) defines:
 *
 *   mx_quantize    Section 3, Algorithm 1: scalar floats -> MX blocks
 *   mx_dequantize  Section 2: v_i = X * P_i, NaN if X is NaN
 *   mx_gemm        Section 4.1 ("Compute Flow"): dot products of two MX operands,
 *                  scalar-float (FP32) output
 *
 * An MX block is k = 32 elements P_i that share one E8M0 scale X = 2^(byte-127)
 * (Section 2, Table 1).  Element formats: FP8 E4M3 / E5M2, FP6 E3M2 / E2M3,
 * FP4 E2M1 and INT8 (Table 1).
 *
 * Conventions common to every entry point
 *   - All data pointers are DEVICE pointers unless the function name ends in
 *     "_host".  The caller allocates and frees every buffer; the library
 *     allocates no device memory.  Shapes and sizes are passed by value or as
 *     HOST arrays.
 *   - Calls are asynchronous on opts->stream (a cudaStream_t passed as void*;
 *     NULL = the legacy default stream).  The "_host" variants synchronise the
 *     stream before they return.
 *   - Return value: MX_OK (0) or a negative mx_status_t.  Nothing throws,
 *     aborts or traps.  mx_strerror() gives a static description;
 *     mx_last_cuda_error() gives the text of the CUDA error behind the last
 *     MX_ERR_CUDA (or which device-side wait expired, after MX_ERR_TIMEOUT) on
 *     the calling thread.
 *   - If the CUDA driver or a GPU is missing every compute entry point returns
 *     MX_ERR_CUDA.  There is no CPU fallback.
 */
#ifndef MX_H_
#define MX_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Element data formats (Table 1).  INT8 is two's complement with value n/64. */
typedef enum {
  MX_E4M3 = 0, /* FP8, 4 exponent / 3 mantissa bits, max normal 448     */
  MX_E5M2 = 1, /* FP8, 5 / 2, max normal 57344                           */
  MX_E3M2 = 2, /* FP6, 3 / 2, max normal 28                              */
  MX_E2M3 = 3, /* FP6, 2 / 3, max normal 7.5                             */
  MX_E2M1 = 4, /* FP4, 2 / 1, max normal 6                               */
  MX_INT8 = 5  /* 1 sign + 1 integer + 6 fraction bits, max 127/64       */
} mx_fmt_t;

/* Rounding of V_i / X onto the element grid (the element cast of Algorithm 1).
 * Section 4.3 uses round-half-to-even for inference, Section 4.5
 * round-half-away-from-zero for training. */
typedef enum { MX_RNE = 0, MX_RHAZ = 1 } mx_round_t;

/* Scalar float type of the unquantized tensor. */
typedef enum { MX_F32 = 0, MX_BF16 = 1 } mx_dtype_t;

/* Where the scale byte of (row, kblock) lives.  Section 2 leaves the layout of
 * a block free; this library keeps scales in their own tensor.
 *   LINEAR   : scales[row * kblocks + kblock]
 *   SWIZZLED : 512-byte chunks of 128 rows x 4 kblocks, the unit one
 *              shared-memory -> tensor-memory copy feeds to the block-scaled
 *              MMA.  See mx_scale_offset().  Padding bytes are written as 0. */
typedef enum { MX_SCALES_LINEAR = 0, MX_SCALES_SWIZZLED = 1 } mx_scale_layout_t;

typedef enum {
  MX_OK = 0,
  MX_ERR_NULL = -1,        /* a required pointer is NULL                     */
  MX_ERR_SHAPE = -2,       /* bad ndim / axis / extent (see each function)   */
  MX_ERR_FMT = -3,         /* enum value out of range                        */
  MX_ERR_ALIGN = -4,       /* a pointer is not aligned as required           */
  MX_ERR_UNSUPPORTED = -5, /* valid request this build does not implement    */
  MX_ERR_CUDA = -6,        /* CUDA runtime / driver error                    */
  MX_ERR_TIMEOUT = -7,     /* a bounded device-side wait gave up             */
  MX_ERR_WORKSPACE = -8    /* caller-supplied workspace is too small         */
} mx_status_t;

/* Optional arguments.  A NULL pointer means
 * { MX_F32, MX_SCALES_SWIZZLED, NULL stream, check_status = 0, pad_k128 = 0 }. */
typedef struct {
  int32_t dtype;        /* mx_dtype_t of the float tensor (input of quantize,
                           output of dequantize); ignored by mx_gemm          */
  int32_t scale_layout; /* mx_scale_layout_t of every scale tensor in the call */
  void* stream;         /* cudaStream_t                                        */
  int32_t check_status; /* mx_gemm, and the mx_quantize / mx_quantize_dual calls that run a
                           tile kernel: nonzero = synchronise the stream and return
                           MX_ERR_TIMEOUT if a device-side wait expired        */
  int32_t pad_k128;     /* 0 or 1.  1: MX tensors are stored as those of the float
                           tensor zero-extended along the block axis to a multiple
                           of 128 elements (zero codes under scale byte 0, which
                           add nothing to a dot product).  mx_quantize writes such
                           tensors -- sizes: mx_elems_bytes / mx_scales_bytes of the
                           shape with shape[axis] rounded up to 128 -- and mx_gemm,
                           mx_gemm_bf16, mx_gemm_ex read them, which lifts the
                           K % 128 rule of 6- and 4-bit operands to K % 32 == 0.
                           Every other entry point returns MX_ERR_UNSUPPORTED for 1;
                           other values: MX_ERR_FMT.                            */
} mx_opts_t;

/* ------------------------------------------------------------------------- */
/* Size and index helpers (host only, no CUDA calls)                         */
/* ------------------------------------------------------------------------- */

/* Bits per element code: 8, 6 or 4; 0 for an invalid format. */
int mx_fmt_bits(mx_fmt_t fmt);

/* Bytes of the packed element tensor produced by mx_quantize for a float tensor
 * of shape[ndim] quantized along `axis`: rows * Lp * bits / 8 with rows = numel /
 * shape[axis] and Lp = shape[axis] rounded up to a multiple of 32 (a partial last
 * block is stored padded, see mx_quantize).  0 on bad arguments. */
size_t mx_elems_bytes(const int64_t* shape, int ndim, int axis, mx_fmt_t fmt);

/* Bytes of the scale tensor for the same call.  rows = numel / shape[axis],
 * kblocks = ceil(shape[axis] / 32).  LINEAR: rows * kblocks.
 * SWIZZLED: ceil(rows/128) * ceil(kblocks/4) * 512.  0 on bad arguments. */
size_t mx_scales_bytes(const int64_t* shape, int ndim, int axis, mx_scale_layout_t layout);

/* Byte offset of the scale of (row, kblock) inside a scale tensor of
 * rows x kblocks.  SWIZZLED:
 *   ((row/128) * ceil(kblocks/4) + kblock/4) * 512
 *     + (row%32)*16 + ((row%128)/32)*4 + kblock%4
 * Returns (size_t)-1 on out-of-range arguments. */
size_t mx_scale_offset(int64_t row, int64_t kblock, int64_t rows, int64_t kblocks,
                       mx_scale_layout_t layout);

const char* mx_strerror(int status);
const char* mx_last_cuda_error(void);

/* ------------------------------------------------------------------------- */
/* mx_quantize -- Algorithm 1 (Section 3)                                    */
/* ------------------------------------------------------------------------- */
/*
 * in         contiguous row-major float tensor of shape[ndim] (opts->dtype),
 *            16-byte aligned.  View it as [outer, L, inner] with
 *            L = shape[axis].  When L is not a multiple of 32 the axis ends in a
 *            partial block: the paper only ever shows whole blocks, and this
 *            library takes the missing elements as +0 (they cannot change the
 *            block maximum) and stores every row padded with zero codes to
 *            Lp = 32 * ceil(L / 32) elements, so that a padded row is again a
 *            valid K-major operand (K = Lp) for mx_gemm.  Such shapes run on a
 *            plain, slower kernel.
 * axis       the axis the scale is shared along (Section 3, last paragraph:
 *            normally the reduction dimension of the matmul that consumes the
 *            tensor).  Block (o, j, b) is in[o, 32b .. 32b+31, j].
 * elems_out  packed element codes, ALWAYS with the quantization axis innermost
 *            ("K-major"): logical [outer*inner, Lp], output row o*inner + j.
 *            For axis == ndim-1 nothing moves; for a 2-D [K x N] tensor with
 *            axis == 0 the result is the [N x K] operand that dgrad / wgrad
 *            need (Section 3: quantizing and transposing do not commute, so
 *            this is a separate tensor; Section 4.1).
 *            Codes form a little-endian bit stream along a row: code i occupies
 *            bits [w*i, w*i + w), w = 8 / 6 / 4.  16-byte aligned,
 *            mx_elems_bytes() long.
 * scales_out one E8M0 byte per block, mx_scales_bytes() long, layout
 *            opts->scale_layout; every byte of the buffer is written.
 *            16-byte aligned.
 *
 * Per block: inputs whose FP32 exponent field is 0 count as signed zero
 * (Section 3, note on subnormals); shared_exp = floor(log2(max|V_i|)) -
 * emax_elem, clamped to [-127, 127]; an all-zero block gets scale byte 0x00; a
 * block holding Inf or NaN gets scale byte 0xFF (X = NaN) and zero codes;
 * P_i = V_i / X rounded (rounding) to the element grid, subnormals included,
 * and saturated to +-max normal with the sign kept (the element cast of Algorithm 1 and its
 * note).  Results that round to zero keep their sign bit in the FP formats.
 *
 * Errors: MX_ERR_NULL, MX_ERR_SHAPE (ndim < 1 or > 8, axis out of range,
 * an extent < 0), MX_ERR_FMT, MX_ERR_ALIGN,
 * MX_ERR_CUDA.  A tensor with zero elements is a successful no-op.
 */
int mx_quantize(const void* in, void* elems_out, uint8_t* scales_out,
                const int64_t* shape, int ndim, int axis,
                mx_fmt_t fmt, mx_round_t rounding, const mx_opts_t* opts);

/*
 * mx_quantize_dual -- both MX tensors of a 2-D tensor in one pass (Sections 3 and 4.1)
 *
 * The training flow of Section 4.1 needs every matmul input quantized along its own reduction
 * axis: X enters Y = X W with blocks along its rows and dW = X^T dY with blocks along its columns,
 * and by Section 3 those are two different MX tensors.  This call reads in[R x C] once and writes
 *   elems_row / scales_row : exactly what mx_quantize(in, axis = 1) writes  ([R x C], K = C)
 *   elems_col / scales_col : exactly what mx_quantize(in, axis = 0) writes  ([C x R], K = R)
 * with the same format, rounding, dtype and scale layout for both.
 * Requirements: R a multiple of 128; C a multiple of 128 (BF16) or 64 (FP32); all pointers
 * 16-byte aligned.  Other shapes: MX_ERR_UNSUPPORTED (call mx_quantize twice instead).
 * Errors otherwise as mx_quantize.
 */
int mx_quantize_dual(const void* in, void* elems_row, uint8_t* scales_row,
                     void* elems_col, uint8_t* scales_col, int64_t R, int64_t C,
                     mx_fmt_t fmt, mx_round_t rounding, const mx_opts_t* opts);

/* ------------------------------------------------------------------------- */
/* mx_dequantize -- Section 2 value semantics                                */
/* ------------------------------------------------------------------------- */
/*
 * elems, scales  an MX tensor as mx_quantize writes it (K-major).
 * shape, ndim    logical float shape of that K-major tensor; axis must be
 *                ndim-1 (anything else: MX_ERR_UNSUPPORTED).  shape[axis] need not
 *                be a multiple of 32: the packed rows are then the padded ones
 *                mx_quantize writes, the output rows are not padded.
 * out            contiguous float tensor of that shape (opts->dtype), 16-byte
 *                aligned.
 * v = decode(P) * 2^(byte-127); scale byte 0xFF -> NaN for the whole block;
 * element codes that encode NaN / Inf (E4M3 0x7F/0xFF; E5M2 0x7C-0x7F and
 * 0xFC-0xFF) decode to NaN / +-Inf; |v| beyond the FP32 range -> +-Inf (the
 * paper leaves that case implementation-defined).  BF16 output rounds to nearest even.
 */
int mx_dequantize(const void* elems, const uint8_t* scales, void* out,
                  const int64_t* shape, int ndim, int axis,
                  mx_fmt_t fmt, const mx_opts_t* opts);

/* ------------------------------------------------------------------------- */
/* mx_gemm -- dot products of MX operands (Section 4.1)                      */
/* ------------------------------------------------------------------------- */
/*
 * A   packed [M x K] codes, K-major (fmtA);  sA its scales, rows = M.
 * B   packed [N x K] codes, K-major (fmtB);  sB its scales, rows = N.
 *     Scales must be in MX_SCALES_SWIZZLED layout with kblocks = K / 32.
 * C   FP32 row-major [M x N], overwritten:
 *       C[m,n] = sum over K-blocks b of X_A[m,b] * X_B[n,b] *
 *                sum_{i<32} P_A[m,32b+i] * P_B[n,32b+i]
 *     accumulated in FP32 on the tensor cores.
 * Shapes: any M >= 0; K a nonzero multiple of 32 (the block size), of 128 when an
 * operand has 6- or 4-bit codes; N such that a row of C is a whole number of 16-byte
 * units (N % 4 for FP32).  Partial tiles are zero-filled on the way in and clipped on
 * the way out; the scale tensors are the padded SWIZZLED tensors mx_quantize writes
 * (padding bytes 0).  A, B 32-byte aligned, sA, sB, C 16-byte aligned.  MX_INT8 operands: MX_ERR_UNSUPPORTED
 * (the block-scaled tensor-core instruction has no integer element type; use
 * mx_gemm_dense).  Products with M <= 96 take a kernel that puts B on the M side of the
 * MMA; its results are bit-identical to the tiled kernels'.
 * Errors: MX_ERR_NULL, MX_ERR_SHAPE, MX_ERR_FMT, MX_ERR_ALIGN,
 * MX_ERR_UNSUPPORTED, MX_ERR_CUDA, MX_ERR_TIMEOUT (only with
 * opts->check_status).
 */
int mx_gemm(const void* A, const uint8_t* sA, const void* B, const uint8_t* sB, float* C,
            int64_t M, int64_t N, int64_t K, mx_fmt_t fmtA, mx_fmt_t fmtB,
            const mx_opts_t* opts);

/*
 * mx_gemm with the result stored as BF16, the scalar-float format the paper keeps
 * tensors in between MX operations (Section 6.2).  C is BF16 row-major [M x N]; each
 * dot product is accumulated in FP32 exactly as in mx_gemm and rounded to nearest even
 * once, in the epilogue.  Requirements and errors are those of mx_gemm.
 */
int mx_gemm_bf16(const void* A, const uint8_t* sA, const void* B, const uint8_t* sB, void* C,
                 int64_t M, int64_t N, int64_t K, mx_fmt_t fmtA, mx_fmt_t fmtB,
                 const mx_opts_t* opts);

/*
 * mx_gemm / mx_gemm_bf16 with the kernel selection and the device-side wait budget in the caller's
 * hands (Section 4.1 defines the product; this call adds nothing to it).  It exists for tuning, for
 * tests that must reach a particular kernel variant, and for the failure drill below; a NULL plan,
 * or a field left at its "library's choice" value, gives exactly mx_gemm.
 *   c_dtype         MX_F32 (C is float*) or MX_BF16.
 *   tile_n          0 = library's choice; 256 or 384 pins the tile width of the two-CTA kernel
 *                   (with 0 a last, less than half full round of 256-wide tiles is computed in
 *                   halves of 128 columns; results do not depend on it).
 *   few_rows_limit  -1 = library's choice (96); 0..128 = largest M that takes the kernel that puts
 *                   B on the M side of the MMA (0 sends every product through the tiled kernels).
 *   wait_cycles     0 = library's choice (about one second); otherwise the budget, in SM clock
 *                   cycles, after which a device-side wait for one pipeline stage gives up (waits
 *                   for a whole tile get four times as much).  When a wait gives up the kernel
 *                   records which one, every warp leaves through the common exit, tensor memory is
 *                   released and the context stays usable; the call (with opts->check_status) or
 *                   the next checked call returns MX_ERR_TIMEOUT and the output is undefined.
 *   drop_fill       -1 = off.  Failure drill: the operand producer leaves out the pipeline fill
 *                   with this running number (0 = the first K chunk of the CTA's first tile): no
 *                   copy is issued for it, so nothing is in flight when the kernel gives up, and
 *                   the MMA issuer's wait for that stage runs out.  Use with a small wait_cycles.
 * Errors as mx_gemm; MX_ERR_FMT for a bad c_dtype, MX_ERR_SHAPE for a field out of range.
 */
typedef struct {
  int32_t c_dtype;
  int32_t tile_n;
  int32_t few_rows_limit;
  int32_t drop_fill;
  int64_t wait_cycles;
} mx_gemm_plan_t;
int mx_gemm_ex(const void* A, const uint8_t* sA, const void* B, const uint8_t* sB, void* C,
               int64_t M, int64_t N, int64_t K, mx_fmt_t fmtA, mx_fmt_t fmtB,
               const mx_opts_t* opts, const mx_gemm_plan_t* plan);

/*
 * `batch` independent products in one launch: the matmuls of attention (scores, context)
 * are dot products like any other (Section 4.1 counts every dot-product operation).
 * A is the packed [batch x M x K] tensor, B [batch x N x K], C [batch x M x N] (c_dtype:
 * MX_F32 or MX_BF16), all contiguous; sA / sB are the swizzled scale tensors of the
 * [batch*M x K] and [batch*N x K] matrices, i.e. what mx_quantize writes for the
 * 3-D tensors along their last axis.  C[b] = A[b] . B[b]^T as in mx_gemm.
 * Requirements and errors as mx_gemm, except that M and N must be multiples of 128 (which
 * keeps every matrix of the stack on whole scale chunks and tiles); additionally MX_ERR_FMT for a bad c_dtype and MX_ERR_SHAPE when
 * batch < 0 or batch*M or batch*N reaches 2^31.  batch == 0 is a no-op.
 */
int mx_gemm_batched(const void* A, const uint8_t* sA, const void* B, const uint8_t* sB, void* C,
                    mx_dtype_t c_dtype, int64_t batch, int64_t M, int64_t N, int64_t K,
                    mx_fmt_t fmtA, mx_fmt_t fmtB, const mx_opts_t* opts);

/*
 * mx_gemm whose epilogue quantizes the result instead of storing it: in the paper's compute
 * flow (Section 4.1) the output of one dot-product operation is requantized to MX before it
 * enters the next one, and when nothing runs in between that pass over C need not touch
 * memory.  Each FP32 accumulator row is cut into blocks of 32 consecutive columns and
 * converted by Algorithm 1 (Section 3) while it is still in registers.
 *   elems_out / scales_out   exactly what mx_quantize(C, shape {M, N}, axis 1, fmtC, rounding)
 *                            writes for the FP32 C that mx_gemm produces from the same
 *                            operands: packed codes [M x N] (N innermost) and the SWIZZLED
 *                            scale tensor of M rows x N/32 blocks -- the A operand of a
 *                            following mx_gemm whose K is this N.  Any format, MX_INT8 included.
 * M and N multiples of 128; elems_out and scales_out 16-byte aligned.  Other requirements
 * and errors as mx_gemm.
 */
int mx_gemm_quantize(const void* A, const uint8_t* sA, const void* B, const uint8_t* sB,
                     void* elems_out, uint8_t* scales_out, int64_t M, int64_t N, int64_t K,
                     mx_fmt_t fmtA, mx_fmt_t fmtB, mx_fmt_t fmtC, mx_round_t rounding,
                     const mx_opts_t* opts);

/*
 * Dot products of MX operands by way of BF16: both operands are dequantized (Section 2) into
 * a caller-supplied DEVICE workspace and multiplied by a dense BF16 tensor-core GEMM with
 * FP32 accumulation.  This is the route for MXINT8 (Table 1), for which the block-scaled
 * tensor-core instruction has no element type, and it accepts every format pair.  The
 * dequantized values are exact in BF16 (an element has at most 7 significant bits, INT8
 * included, and the scale is a power of two) unless X * P falls below BF16's normal range
 * (scale bytes under ~10), so the result obeys the same bound as mx_gemm; it runs at the
 * BF16 rate, half the FP8 one, plus the two dequantize passes.
 *   C          FP32 or BF16 (c_dtype) row-major [M x N].
 *   workspace  at least mx_gemm_dense_workspace_bytes(M, N, K) = 2 (M + N) K bytes (rounded
 *              up to 256 each), 256-byte aligned; contents undefined afterwards.
 * Requirements as mx_gemm except that A and B need 16-byte alignment only, K may be any
 * nonzero multiple of 32 for every format and MX_INT8 is allowed.  Additional errors: MX_ERR_WORKSPACE; MX_ERR_FMT for a bad c_dtype.
 */
size_t mx_gemm_dense_workspace_bytes(int64_t M, int64_t N, int64_t K);
int mx_gemm_dense(const void* A, const uint8_t* sA, const void* B, const uint8_t* sB, void* C,
                  mx_dtype_t c_dtype, int64_t M, int64_t N, int64_t K, mx_fmt_t fmtA, mx_fmt_t fmtB,
                  const mx_opts_t* opts, void* workspace, size_t workspace_bytes);

/* ------------------------------------------------------------------------- */
/* Convolution as a dot product (Section 4.1)                                */
/* ------------------------------------------------------------------------- */
/*
 * The paper counts convolution among the dot-product operations that take MX operands.
 * Here the reduction axis of a 2-D convolution is (kh, kw, C) with the channel innermost,
 * and an MX block is 32 consecutive channels of one filter tap (C % 32 == 0, so no block
 * straddles two taps).  The activation x[N, H, W, C] (channels last) is then quantized ONCE
 * with mx_quantize along C, and mx_im2col lays its codes and scales out as the K-major
 * operand A[M x K] of mx_gemm, M = N*Ho*Wo, K = kh*kw*C; taps that fall into the zero padding
 * become zero blocks (codes 0, scale byte 0).  No value is requantized.  With the filter
 * w[Cout, kh, kw, C] quantized along its last axis (rows = Cout, K = kh*kw*C),
 *     y[N, Ho, Wo, Cout] = mx_gemm(A, w)        (row-major [M x Cout] is channels-last y).
 * Ho = (H + 2 pad_h - dil_h (kh - 1) - 1) / stride_h + 1, Wo likewise.  mx_gemm's own shape rules
 * apply to K = kh*kw*C (a multiple of 128 for 6- and 4-bit codes).
 */
typedef struct {
  int64_t N, H, W, C;          /* activation, channels last                         */
  int32_t kh, kw;              /* filter taps                                       */
  int32_t stride_h, stride_w;  /* >= 1                                              */
  int32_t pad_h, pad_w;        /* zero padding on both sides, >= 0                  */
  int32_t dil_h, dil_w;        /* >= 1                                              */
} mx_conv_t;

/* Output extent of the convolution; 0 on bad arguments. */
int64_t mx_conv_out_h(const mx_conv_t* conv);
int64_t mx_conv_out_w(const mx_conv_t* conv);

/*
 * elems_in, scales_in   MX tensor of x viewed as [N*H*W rows x C] (what mx_quantize writes for
 *                       shape {N, H, W, C}, axis 3); scales in opts->scale_layout.
 * elems_out             packed [M x kh*kw*C] codes, mx_elems_bytes of that shape.
 * scales_out            SWIZZLED scale tensor of M rows x kh*kw*C/32 blocks (padding written 0).
 * Requirements: C % 32 == 0 and C * bits / 8 a multiple of 16 (6-bit codes: C % 64 == 0);
 * all four pointers 16-byte aligned; the output codes below 64 GiB (2^32 16-byte chunks).
 * Errors: MX_ERR_NULL, MX_ERR_SHAPE, MX_ERR_FMT, MX_ERR_ALIGN, MX_ERR_CUDA.
 */
int mx_im2col(const void* elems_in, const uint8_t* scales_in, void* elems_out, uint8_t* scales_out,
              const mx_conv_t* conv, mx_fmt_t fmt, const mx_opts_t* opts);

/*
 * mx_conv2d -- the same convolution without the materialized operand (Section 4.1).
 *
 * Block (m, kb) of the operand mx_im2col would write is a copy of a block of the quantized
 * activation (or zero), so the GEMM kernel can fetch it from there itself: four warps gather each
 * pipeline stage's 128 rows x 128 codes and their scale bytes while the tensor core works on the
 * stages before, and the [M x kh kw C] operand (kh kw times the activation) is never written or
 * read.  The arithmetic is that of mx_im2col + mx_gemm; results obey the same bound.
 *   x_elems, x_scales   MX tensor of x[N, H, W, C] quantized along C (rows N*H*W); scales in
 *                       opts->scale_layout.  MX_E4M3 or MX_E5M2 (one byte per code: the gather copies
 *                       bytes into the tensor core's operand layout; 6- and 4-bit activations:
 *                       MX_ERR_UNSUPPORTED, use mx_im2col + mx_gemm).
 *   w_elems, w_scales   the filter w[Cout, kh, kw, C] quantized along (kh, kw, C) as one axis: packed
 *                       [Cout x kh kw C], SWIZZLED scales.  Any format but MX_INT8; kh*kw*C a
 *                       multiple of 128 for 6- and 4-bit filters.
 *   y                   FP32 or BF16 (y_dtype) [N, Ho, Wo, Cout], channels last.
 * C % 32 == 0; Cout * sizeof(y element) a multiple of 16; x_elems, x_scales, y 16-byte aligned,
 * w_elems 32-byte, w_scales 16-byte aligned.  Errors as mx_gemm and mx_im2col.
 */
int mx_conv2d(const void* x_elems, const uint8_t* x_scales, const void* w_elems, const uint8_t* w_scales,
              void* y, mx_dtype_t y_dtype, const mx_conv_t* conv, int64_t Cout, mx_fmt_t fmt_x,
              mx_fmt_t fmt_w, const mx_opts_t* opts);

/* ------------------------------------------------------------------------- */
/* Host-buffer variants                                                      */
/* ------------------------------------------------------------------------- */
/*
 * Same operations with HOST input and output buffers (pinned memory gives the
 * best copy rate, pageable memory works).  The caller supplies a DEVICE
 * workspace of at least mx_*_host_workspace_bytes(); the call copies the
 * inputs to it, runs the device entry point above, copies the results back and
 * synchronises opts->stream.  Additional error: MX_ERR_WORKSPACE.
 * mx_quantize_host and mx_dequantize_host cut a tensor of 8 MiB or more whose
 * blocks run along its last axis into row chunks and overlap the copies of
 * neighbouring chunks in the two directions of the host link; for that they
 * create, once per device, two streams and a few events of their own (work queued
 * on opts->stream before the call still comes first).
 */
size_t mx_quantize_host_workspace_bytes(const int64_t* shape, int ndim, int axis,
                                        mx_fmt_t fmt, const mx_opts_t* opts);
int mx_quantize_host(const void* in_host, void* elems_out_host, uint8_t* scales_out_host,
                     const int64_t* shape, int ndim, int axis,
                     mx_fmt_t fmt, mx_round_t rounding, const mx_opts_t* opts,
                     void* workspace_dev, size_t workspace_bytes);

/*
 * mx_quantize_host_static -- mx_quantize_host without a caller-supplied workspace.
 * (The paper has no counterpart: this is a deployment convenience of this library.)
 *
 * Some callers of mx_quantize_host cannot provide its device workspace because they are not
 * allowed to allocate device memory at all: a plug-in inside a host application that has
 * handed every free byte of the GPU to its own memory pool and forbids further allocations,
 * or a latency-critical loop that must never enter cudaMalloc (which may synchronise the
 * device).  For them the staging area lives in a fixed array inside the library,
 * MX_STATIC_SCRATCH_BYTES long, which every GPU that loads the library holds from module
 * load until the process exits.  This call allocates nothing: no cudaMalloc, no cudaFree,
 * no allocating library routine.
 *
 * Arguments, results and errors are those of mx_quantize_host (host input, host outputs, the
 * stream is synchronised before returning).  A request whose staging need
 * (mx_quantize_host_workspace_bytes) exceeds MX_STATIC_SCRATCH_BYTES is rejected with
 * MX_ERR_WORKSPACE and nothing is launched.
 *
 * The first call on a device looks up the device address of the array (once per device, with
 * that device current); make that first call outside any stream capture.  All calls on a
 * device share the one array and it keeps the bytes of the previous call: the routine
 * rewrites every byte it later reads back (including the padding of the swizzled scale
 * tensor), but two calls that overlap on the GPU -- from two threads or two streams -- race
 * on it and must be serialised by the caller.
 */
#define MX_STATIC_SCRATCH_BYTES (16u * 1024u * 1024u)
int mx_quantize_host_static(const void* in_host, void* elems_out_host, uint8_t* scales_out_host,
                            const int64_t* shape, int ndim, int axis,
                            mx_fmt_t fmt, mx_round_t rounding, const mx_opts_t* opts);

size_t mx_dequantize_host_workspace_bytes(const int64_t* shape, int ndim, int axis,
                                          mx_fmt_t fmt, const mx_opts_t* opts);
int mx_dequantize_host(const void* elems_host, const uint8_t* scales_host, void* out_host,
                       const int64_t* shape, int ndim, int axis,
                       mx_fmt_t fmt, const mx_opts_t* opts,
                       void* workspace_dev, size_t workspace_bytes);

/*
 * Asynchronous forms of the two calls above, for a sequence of conversions whose copies should
 * overlap ACROSS calls: each returns after queueing its work on the library's internal copy
 * pipeline; calls execute in the order issued, the upload of one call overlapping the download
 * of the one before.  Results (and the host input buffers) may be touched again only after
 * mx_host_synchronize().  Until then every queued call needs its own workspace, and a call must
 * not read host memory that an earlier, still queued call writes.  Blocks must run along the
 * last axis (otherwise MX_ERR_UNSUPPORTED); other arguments and errors as the synchronous forms.
 * mx_host_synchronize waits for everything queued on the current device.
 */
int mx_quantize_host_async(const void* in_host, void* elems_out_host, uint8_t* scales_out_host,
                           const int64_t* shape, int ndim, int axis,
                           mx_fmt_t fmt, mx_round_t rounding, const mx_opts_t* opts,
                           void* workspace_dev, size_t workspace_bytes);
int mx_dequantize_host_async(const void* elems_host, const uint8_t* scales_host, void* out_host,
                             const int64_t* shape, int ndim, int axis,
                             mx_fmt_t fmt, const mx_opts_t* opts,
                             void* workspace_dev, size_t workspace_bytes);
int mx_host_synchronize(void);

size_t mx_gemm_host_workspace_bytes(int64_t M, int64_t N, int64_t K,
                                    mx_fmt_t fmtA, mx_fmt_t fmtB);
int mx_gemm_host(const void* A_host, const uint8_t* sA_host,
                 const void* B_host, const uint8_t* sB_host, float* C_host,
                 int64_t M, int64_t N, int64_t K, mx_fmt_t fmtA, mx_fmt_t fmtB,
                 const mx_opts_t* opts, void* workspace_dev, size_t workspace_bytes);

#ifdef __cplusplus
}
#endif
#endif /* MX_H_ */
