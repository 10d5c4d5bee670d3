// C ABI of the library (declared in include/mx.h): argument validation, size
// helpers, kernel dispatch and the host-buffer variants.  No arithmetic of the
// method lives here.
#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "mx.h"
#include "mx_launch.h"

namespace {

thread_local char g_cuda_error[256] = "";

int fail_cuda(cudaError_t e) {
  std::snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s", cudaGetErrorName(e),
                cudaGetErrorString(e));
  return MX_ERR_CUDA;
}

bool fmt_ok(int f) { return f >= MX_E4M3 && f <= MX_INT8; }
int fmt_bits(int f) {
  switch (f) {
    case MX_E4M3: case MX_E5M2: case MX_INT8: return 8;
    case MX_E3M2: case MX_E2M3: return 6;
    case MX_E2M1: return 4;
    default: return 0;
  }
}

struct View {
  int64_t outer, L, inner, numel, rows, kblocks;
  int64_t Lp;            // L rounded up to whole blocks: the length of a packed row in elements
  int64_t padded_numel;  // rows * Lp
};

// [outer, L, inner] view of shape[ndim] around `axis`; false on a bad shape.  Every product is
// formed with an overflow check and the padded element count is held below 2^44, so that no byte
// count derived from the view (at most 4 bytes per element plus alignment) can wrap a size_t or
// come out smaller than the tensor it describes.
constexpr int64_t kMaxElements = (int64_t)1 << 44;

// pad128: the packed rows (and the scale tensor) are those of the tensor zero-extended along the
// axis to a multiple of 128 elements (mx_opts_t::pad_k128).
bool make_view(const int64_t* shape, int ndim, int axis, View* v, bool pad128 = false) {
  if (!shape || ndim < 1 || ndim > 8 || axis < 0 || axis >= ndim) return false;
  v->outer = v->inner = 1;
  for (int i = 0; i < ndim; ++i) {
    if (shape[i] < 0) return false;
    if (i < axis && __builtin_mul_overflow(v->outer, shape[i], &v->outer)) return false;
    if (i > axis && __builtin_mul_overflow(v->inner, shape[i], &v->inner)) return false;
  }
  v->L = shape[axis];
  if (v->L > kMaxElements) return false;
  v->kblocks = (v->L + 31) / 32;  // a last, partial block is stored padded with zero codes
  if (pad128) v->kblocks = (v->kblocks + 3) / 4 * 4;
  v->Lp = v->kblocks * 32;
  if (__builtin_mul_overflow(v->outer, v->inner, &v->rows)) return false;
  if (__builtin_mul_overflow(v->rows, v->L, &v->numel)) return false;
  if (__builtin_mul_overflow(v->rows, v->Lp, &v->padded_numel)) return false;
  if (v->padded_numel > kMaxElements) return false;
  // the swizzled scale tensor pads rows to 128 and blocks to 4: bounded by 16 x (rows + 128) x (kblocks + 4)
  int64_t sc;
  if (__builtin_mul_overflow(v->rows + 128, v->kblocks + 4, &sc) || sc > kMaxElements) return false;
  return true;
}

size_t scales_bytes(int64_t rows, int64_t kblocks, int layout) {
  if (layout == MX_SCALES_LINEAR) return (size_t)(rows * kblocks);
  return (size_t)(((rows + 127) / 128) * ((kblocks + 3) / 4) * 512);
}

struct Opts {
  int dtype, layout, check, pad128;
  cudaStream_t stream;
};
bool read_opts(const mx_opts_t* o, Opts* out) {
  out->dtype = o ? o->dtype : MX_F32;
  out->layout = o ? o->scale_layout : MX_SCALES_SWIZZLED;
  out->stream = o ? (cudaStream_t)o->stream : nullptr;
  out->check = o ? o->check_status : 0;
  out->pad128 = o ? o->pad_k128 : 0;
  return (out->pad128 == 0 || out->pad128 == 1) && (out->dtype == MX_F32 || out->dtype == MX_BF16) &&
         (out->layout == MX_SCALES_LINEAR || out->layout == MX_SCALES_SWIZZLED);
}

// SM count of the current device, cached per device ordinal.
int sm_count(cudaError_t* err) {
  static int cache[64] = {0};
  int dev = 0;
  *err = cudaGetDevice(&dev);
  if (*err != cudaSuccess) return 0;
  if (dev >= 0 && dev < 64 && cache[dev]) return cache[dev];
  int n = 0;
  *err = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
  if (*err != cudaSuccess) return 0;
  if (dev >= 0 && dev < 64) cache[dev] = n;
  return n;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace

extern "C" {

int mx_fmt_bits(mx_fmt_t fmt) { return fmt_bits((int)fmt); }

size_t mx_elems_bytes(const int64_t* shape, int ndim, int axis, mx_fmt_t fmt) {
  View v;
  if (!fmt_ok((int)fmt) || !make_view(shape, ndim, axis, &v)) return 0;
  return (size_t)(v.padded_numel / 8 * fmt_bits((int)fmt));
}

size_t mx_scales_bytes(const int64_t* shape, int ndim, int axis, mx_scale_layout_t layout) {
  View v;
  if ((layout != MX_SCALES_LINEAR && layout != MX_SCALES_SWIZZLED) ||
      !make_view(shape, ndim, axis, &v))
    return 0;
  return scales_bytes(v.rows, v.kblocks, (int)layout);
}

size_t mx_scale_offset(int64_t row, int64_t kblock, int64_t rows, int64_t kblocks,
                       mx_scale_layout_t layout) {
  if (row < 0 || row >= rows || kblock < 0 || kblock >= kblocks) return (size_t)-1;
  if (layout == MX_SCALES_LINEAR) return (size_t)(row * kblocks + kblock);
  if (layout != MX_SCALES_SWIZZLED) return (size_t)-1;
  const int64_t kchunks = (kblocks + 3) / 4;
  return (size_t)(((row / 128) * kchunks + kblock / 4) * 512 + (row % 32) * 16 +
                  ((row % 128) / 32) * 4 + kblock % 4);
}

const char* mx_strerror(int status) {
  switch (status) {
    case MX_OK: return "ok";
    case MX_ERR_NULL: return "a required pointer is NULL";
    case MX_ERR_SHAPE: return "bad shape, axis or extent";
    case MX_ERR_FMT: return "enum value out of range";
    case MX_ERR_ALIGN: return "pointer not aligned as required";
    case MX_ERR_UNSUPPORTED: return "request not supported by this build";
    case MX_ERR_CUDA: return "CUDA error (see mx_last_cuda_error)";
    case MX_ERR_TIMEOUT: return "a bounded device-side wait gave up";
    case MX_ERR_WORKSPACE: return "workspace too small";
    default: return "unknown status";
  }
}

const char* mx_last_cuda_error(void) { return g_cuda_error; }

// After a launch of one of the tile kernels with opts->check_status: synchronise the stream and
// report a bounded device-side wait that gave up.
static int tile_status_check(cudaStream_t stream) {
  unsigned int st = 0;
  const cudaError_t e = mx::quantize_tile_status(stream, &st);
  if (e != cudaSuccess) return fail_cuda(e);
  if (st != 0) {
    std::snprintf(g_cuda_error, sizeof(g_cuda_error), "device-side wait %u of a tile kernel gave up "
                  "(1 a tile's copy never landed, 2 a stage was never released)", st);
    return MX_ERR_TIMEOUT;
  }
  return MX_OK;
}

int mx_quantize(const void* in, void* elems_out, uint8_t* scales_out, const int64_t* shape,
                int ndim, int axis, mx_fmt_t fmt, mx_round_t rounding, const mx_opts_t* opts) {
  Opts o;
  View v;
  if (!shape) return MX_ERR_NULL;
  if (!fmt_ok((int)fmt) || (rounding != MX_RNE && rounding != MX_RHAZ) || !read_opts(opts, &o))
    return MX_ERR_FMT;
  if (!make_view(shape, ndim, axis, &v, o.pad128 != 0)) return MX_ERR_SHAPE;
  if (v.numel == 0) return MX_OK;
  if (!in || !elems_out || !scales_out) return MX_ERR_NULL;
  if ((uintptr_t)in % 16 || (uintptr_t)elems_out % 16 || (uintptr_t)scales_out % 16)
    return MX_ERR_ALIGN;
  if (v.padded_numel / 8 >= (int64_t)1 << 31 || v.rows >= (int64_t)1 << 31 || v.inner >= (int64_t)1 << 31 ||
      v.L >= (int64_t)1 << 31)
    return MX_ERR_UNSUPPORTED;
  cudaError_t e;
  mx::QuantizeArgs a;
  a.in = in; a.elems = (uint8_t*)elems_out; a.scales = scales_out;
  a.outer = v.outer; a.L = v.L; a.L_store = v.Lp; a.inner = v.inner; a.numel = v.numel;
  a.fmt = (int)fmt; a.rounding = (int)rounding; a.dtype = o.dtype; a.layout = o.layout;
  a.stream = o.stream;
  a.sm_count = sm_count(&e);
  if (e != cudaSuccess) return fail_cuda(e);
  // The swizzled tensor has padding when rows % 128 or kblocks % 4 is nonzero:
  // zero the buffer first so that every byte is defined.
  if (o.layout == MX_SCALES_SWIZZLED && (v.rows % 128 != 0 || v.kblocks % 4 != 0)) {
    e = cudaMemsetAsync(scales_out, 0, scales_bytes(v.rows, v.kblocks, o.layout), o.stream);
    if (e != cudaSuccess) return fail_cuda(e);
  }
  // Axis 0 of a 2-D BF16 tensor of whole 128 x 128 tiles, 6- or 4-bit codes: the tile kernel's column
  // pass (its copies in flight cost no registers; the register kernels are request-bound at the
  // occupancy their staged variants have)
  if (o.dtype == MX_BF16 && fmt_bits((int)fmt) != 8 && v.outer == 1 && v.inner > 1 && v.L % 128 == 0 &&
      v.inner % 128 == 0 && v.Lp == v.L) {
    mx::DualArgs d;
    d.in = in; d.elems_row = nullptr; d.scales_row = nullptr;
    d.elems_col = (uint8_t*)elems_out; d.scales_col = scales_out;
    d.R = v.L; d.C = v.inner; d.fmt = (int)fmt; d.rounding = (int)rounding; d.dtype = o.dtype; d.layout = o.layout;
    d.sm_count = a.sm_count; d.stream = o.stream;
    e = mx::launch_quantize_tile_cols(d);
    if (e != cudaSuccess) return fail_cuda(e);
    return o.check ? tile_status_check(o.stream) : MX_OK;
  }
  e = mx::launch_quantize(a);
  return e == cudaSuccess ? MX_OK : fail_cuda(e);
}

int mx_quantize_dual(const void* in, void* elems_row, uint8_t* scales_row, void* elems_col,
                     uint8_t* scales_col, int64_t R, int64_t C, mx_fmt_t fmt, mx_round_t rounding,
                     const mx_opts_t* opts) {
  Opts o;
  if (!fmt_ok((int)fmt) || (rounding != MX_RNE && rounding != MX_RHAZ) || !read_opts(opts, &o))
    return MX_ERR_FMT;
  if (o.pad128) return MX_ERR_UNSUPPORTED;  // zero-extended rows: mx_quantize and mx_gemm* only
  if (R < 0 || C < 0 || R % 32 || C % 32) return MX_ERR_SHAPE;
  if (R == 0 || C == 0) return MX_OK;
  if (!in || !elems_row || !scales_row || !elems_col || !scales_col) return MX_ERR_NULL;
  if ((uintptr_t)in % 16 || (uintptr_t)elems_row % 16 || (uintptr_t)scales_row % 16 ||
      (uintptr_t)elems_col % 16 || (uintptr_t)scales_col % 16)
    return MX_ERR_ALIGN;
  const int64_t strip = o.dtype == MX_BF16 ? 128 : 64;
  if (R % 128 || C % strip || R >= ((int64_t)1 << 31) || C >= ((int64_t)1 << 31)) return MX_ERR_UNSUPPORTED;
  mx::DualArgs a;
  a.in = in;
  a.elems_row = (uint8_t*)elems_row; a.scales_row = scales_row;
  a.elems_col = (uint8_t*)elems_col; a.scales_col = scales_col;
  a.R = R; a.C = C; a.fmt = (int)fmt; a.rounding = (int)rounding; a.dtype = o.dtype; a.layout = o.layout;
  a.stream = o.stream;
  cudaError_t e;
  a.sm_count = sm_count(&e);
  if (e != cudaSuccess) return fail_cuda(e);
  // swizzled scale tensors have padding when kblocks % 4 != 0 (rows are multiples of 128 here)
  if (o.layout == MX_SCALES_SWIZZLED && (C / 32) % 4 != 0) {
    e = cudaMemsetAsync(scales_row, 0, scales_bytes(R, C / 32, o.layout), o.stream);
    if (e != cudaSuccess) return fail_cuda(e);
  }
  if (o.layout == MX_SCALES_SWIZZLED && C % 128 != 0) {  // rows of the [C x R] scale tensor
    e = cudaMemsetAsync(scales_col, 0, scales_bytes(C, R / 32, o.layout), o.stream);
    if (e != cudaSuccess) return fail_cuda(e);
  }
  // BF16: tiles through shared memory (TMA); FP32: the register kernel, except 6-bit codes of whole
  // 128 x 128 tiles, which take a tile kernel too (the register kernel's staged variants are the slow ones)
  const bool f32_tiles = o.dtype == MX_F32 && (fmt == MX_E3M2 || fmt == MX_E2M3) && C % 128 == 0;
  e = o.dtype == MX_BF16 ? mx::launch_quantize_tile(a) : f32_tiles ? mx::launch_quantize_tile_f32(a)
                                                                   : mx::launch_quantize_dual(a);
  if (e != cudaSuccess) return fail_cuda(e);
  return (o.check && (o.dtype == MX_BF16 || f32_tiles)) ? tile_status_check(o.stream) : MX_OK;
}

int mx_dequantize(const void* elems, const uint8_t* scales, void* out, const int64_t* shape,
                  int ndim, int axis, mx_fmt_t fmt, const mx_opts_t* opts) {
  Opts o;
  View v;
  if (!shape) return MX_ERR_NULL;
  if (!fmt_ok((int)fmt) || !read_opts(opts, &o)) return MX_ERR_FMT;
  if (o.pad128) return MX_ERR_UNSUPPORTED;  // zero-extended rows: mx_quantize and mx_gemm* only
  if (!make_view(shape, ndim, axis, &v)) return MX_ERR_SHAPE;
  if (axis != ndim - 1) return MX_ERR_UNSUPPORTED;
  if (v.numel == 0) return MX_OK;
  if (!elems || !scales || !out) return MX_ERR_NULL;
  if ((uintptr_t)elems % 16 || (uintptr_t)scales % 16 || (uintptr_t)out % 16) return MX_ERR_ALIGN;
  if (v.padded_numel / 8 >= (int64_t)1 << 31 || v.L >= (int64_t)1 << 31) return MX_ERR_UNSUPPORTED;
  cudaError_t e;
  mx::DequantizeArgs a;
  a.elems = (const uint8_t*)elems; a.scales = scales; a.out = out;
  a.rows = v.rows; a.L = v.L; a.fmt = (int)fmt; a.dtype = o.dtype; a.layout = o.layout;
  a.stream = o.stream;
  a.sm_count = sm_count(&e);
  if (e != cudaSuccess) return fail_cuda(e);
  e = mx::launch_dequantize(a);
  return e == cudaSuccess ? MX_OK : fail_cuda(e);
}

// ---------------------------------------------------------------------------
// Host-buffer variants: copy in, run the device entry point, copy out, sync.
// ---------------------------------------------------------------------------

size_t mx_quantize_host_workspace_bytes(const int64_t* shape, int ndim, int axis, mx_fmt_t fmt,
                                        const mx_opts_t* opts) {
  Opts o;
  View v;
  if (!fmt_ok((int)fmt) || !read_opts(opts, &o) || !make_view(shape, ndim, axis, &v)) return 0;
  const size_t in_b = (size_t)v.numel * (o.dtype == MX_BF16 ? 2 : 4);
  return align_up(in_b, 256) + align_up((size_t)v.padded_numel / 8 * fmt_bits((int)fmt), 256) +
         align_up(scales_bytes(v.rows, v.kblocks, o.layout), 256);
}

}  // extern "C"

namespace {

// Two internal streams and a few events per device for the host-buffer entry points: a tensor
// whose blocks run along the last axis is cut into row chunks (multiples of 128 rows, so every
// chunk owns whole pieces of the packed tensor and of either scale layout); chunk i + 1 travels to
// the device while chunk i is converted and chunk i - 1 travels back, which keeps both directions
// of the host link busy instead of one after the other.
constexpr int kMaxChunks = 4;                // measured: 3 to 8 chunks differ by a few per cent
constexpr size_t kMinChunkBytes = 4u << 20;  // of float data; below this the copies are latency-bound

struct HostPipe {
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t start = nullptr, done[kMaxChunks] = {};
  bool ready = false;
};

HostPipe* host_pipe(cudaError_t* err) {
  static HostPipe pipes[64];
  int dev = 0;
  *err = cudaGetDevice(&dev);
  if (*err != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  HostPipe* p = &pipes[dev];
  if (p->ready) return p;
  if ((*err = cudaStreamCreateWithFlags(&p->in, cudaStreamNonBlocking)) != cudaSuccess) return nullptr;
  if ((*err = cudaStreamCreateWithFlags(&p->out, cudaStreamNonBlocking)) != cudaSuccess) return nullptr;
  if ((*err = cudaEventCreateWithFlags(&p->start, cudaEventDisableTiming)) != cudaSuccess) return nullptr;
  for (int i = 0; i < kMaxChunks; ++i)
    if ((*err = cudaEventCreateWithFlags(&p->done[i], cudaEventDisableTiming)) != cudaSuccess) return nullptr;
  p->ready = true;
  return p;
}

// Rows per chunk (a multiple of 128) and the number of chunks; 1 chunk = do not pipeline.
int plan_chunks(int64_t rows, size_t float_bytes, int64_t* rows_per_chunk) {
  int n = (int)(float_bytes / kMinChunkBytes);
  if (n > kMaxChunks) n = kMaxChunks;
  if (n < 2 || rows < 256) { *rows_per_chunk = rows; return 1; }
  int64_t rpc = (rows + n - 1) / n;
  rpc = (rpc + 127) / 128 * 128;
  *rows_per_chunk = rpc;
  return (int)((rows + rpc - 1) / rpc);
}

// Byte offset of the scales of row r0 (a multiple of 128) in either layout.
size_t scales_row_offset(int64_t r0, int64_t kblocks, int layout) {
  return layout == MX_SCALES_LINEAR ? (size_t)r0 * (size_t)kblocks
                                    : (size_t)(r0 / 128) * (size_t)((kblocks + 3) / 4) * 512;
}

int quantize_host_impl(const void* in_host, void* elems_out_host, uint8_t* scales_out_host,
                       const int64_t* shape, int ndim, int axis, mx_fmt_t fmt, mx_round_t rounding,
                       const mx_opts_t* opts, void* workspace_dev, size_t workspace_bytes,
                       bool may_pipeline, bool async = false) {
  Opts o;
  View v;
  if (!shape) return MX_ERR_NULL;
  if (!fmt_ok((int)fmt) || !read_opts(opts, &o)) return MX_ERR_FMT;
  if (o.pad128) return MX_ERR_UNSUPPORTED;  // zero-extended rows: mx_quantize and mx_gemm* only
  if (!make_view(shape, ndim, axis, &v)) return MX_ERR_SHAPE;
  if (v.numel == 0) return MX_OK;
  if (!in_host || !elems_out_host || !scales_out_host || !workspace_dev) return MX_ERR_NULL;
  if ((uintptr_t)workspace_dev % 256) return MX_ERR_ALIGN;
  if (workspace_bytes < mx_quantize_host_workspace_bytes(shape, ndim, axis, fmt, opts))
    return MX_ERR_WORKSPACE;
  const size_t esz = o.dtype == MX_BF16 ? 2 : 4;
  const size_t in_b = (size_t)v.numel * esz;
  const size_t el_b = (size_t)v.padded_numel / 8 * fmt_bits((int)fmt);
  const size_t sc_b = scales_bytes(v.rows, v.kblocks, o.layout);
  char* d_in = (char*)workspace_dev;
  char* d_el = d_in + align_up(in_b, 256);
  char* d_sc = d_el + align_up(el_b, 256);
  cudaError_t e;
  int64_t rpc = v.rows;
  const int chunks = (may_pipeline && axis == ndim - 1) ? plan_chunks(v.rows, in_b, &rpc) : 1;
  if (async && axis != ndim - 1) return MX_ERR_UNSUPPORTED;
  if (chunks > 1 || async) {
    HostPipe* hp = host_pipe(&e);
    if (!hp) return fail_cuda(e);
    // work queued on the caller's stream comes first
    if ((e = cudaEventRecord(hp->start, o.stream)) != cudaSuccess ||
        (e = cudaStreamWaitEvent(hp->in, hp->start, 0)) != cudaSuccess ||
        (e = cudaStreamWaitEvent(hp->out, hp->start, 0)) != cudaSuccess)
      return fail_cuda(e);
    mx_opts_t co = {o.dtype, o.layout, hp->in, 0};
    const size_t row_in = (size_t)v.L * esz, row_el = (size_t)v.Lp / 8 * fmt_bits((int)fmt);
    for (int c = 0; c < chunks; ++c) {
      const int64_t r0 = c * rpc, nr = (r0 + rpc <= v.rows ? rpc : v.rows - r0);
      const size_t so = scales_row_offset(r0, v.kblocks, o.layout);
      const size_t sb = scales_bytes(nr, v.kblocks, o.layout);
      if ((e = cudaMemcpyAsync(d_in + r0 * row_in, (const char*)in_host + r0 * row_in, nr * row_in,
                               cudaMemcpyHostToDevice, hp->in)) != cudaSuccess)
        return fail_cuda(e);
      const int64_t cshape[2] = {nr, v.L};
      const int rc = mx_quantize(d_in + r0 * row_in, d_el + r0 * row_el, (uint8_t*)d_sc + so, cshape, 2, 1, fmt,
                                 rounding, &co);
      if (rc != MX_OK) return rc;
      if ((e = cudaEventRecord(hp->done[c], hp->in)) != cudaSuccess ||
          (e = cudaStreamWaitEvent(hp->out, hp->done[c], 0)) != cudaSuccess ||
          (e = cudaMemcpyAsync((char*)elems_out_host + r0 * row_el, d_el + r0 * row_el, nr * row_el,
                               cudaMemcpyDeviceToHost, hp->out)) != cudaSuccess)
        return fail_cuda(e);
      (void)sb;
    }
    // the scale tensor is small: one copy after the last chunk
    if ((e = cudaMemcpyAsync(scales_out_host, d_sc, sc_b, cudaMemcpyDeviceToHost, hp->out)) != cudaSuccess)
      return fail_cuda(e);
    if (async) return MX_OK;  // mx_host_synchronize() waits for it
    if ((e = cudaStreamSynchronize(hp->out)) != cudaSuccess || (e = cudaStreamSynchronize(hp->in)) != cudaSuccess ||
        (e = cudaStreamSynchronize(o.stream)) != cudaSuccess)
      return fail_cuda(e);
    return MX_OK;
  }
  e = cudaMemcpyAsync(d_in, in_host, in_b, cudaMemcpyHostToDevice, o.stream);
  if (e != cudaSuccess) return fail_cuda(e);
  const int rc = mx_quantize(d_in, d_el, (uint8_t*)d_sc, shape, ndim, axis, fmt, rounding, opts);
  if (rc != MX_OK) return rc;
  e = cudaMemcpyAsync(elems_out_host, d_el, el_b, cudaMemcpyDeviceToHost, o.stream);
  if (e != cudaSuccess) return fail_cuda(e);
  e = cudaMemcpyAsync(scales_out_host, d_sc, sc_b, cudaMemcpyDeviceToHost, o.stream);
  if (e != cudaSuccess) return fail_cuda(e);
  e = cudaStreamSynchronize(o.stream);
  return e == cudaSuccess ? MX_OK : fail_cuda(e);
}

}  // namespace

extern "C" {

int mx_quantize_host(const void* in_host, void* elems_out_host, uint8_t* scales_out_host,
                     const int64_t* shape, int ndim, int axis, mx_fmt_t fmt, mx_round_t rounding,
                     const mx_opts_t* opts, void* workspace_dev, size_t workspace_bytes) {
  return quantize_host_impl(in_host, elems_out_host, scales_out_host, shape, ndim, axis, fmt, rounding, opts,
                            workspace_dev, workspace_bytes, true);
}

// ---------------------------------------------------------------------------
// Host-buffer quantize for callers that may not allocate device memory
// ---------------------------------------------------------------------------

}  // extern "C"

namespace {

// Staging area of mx_quantize_host_static.  In host code this name is only a handle for the
// symbol, not a device address: the address is looked up once per device below.
static __device__ __align__(256) unsigned char g_static_scratch[MX_STATIC_SCRATCH_BYTES];

// Device address of g_static_scratch on the current device (cached per device ordinal).
void* static_scratch_address(cudaError_t* err) {
  static void* cache[64] = {nullptr};
  int dev = 0;
  *err = cudaGetDevice(&dev);
  if (*err != cudaSuccess) return nullptr;
  if (dev >= 0 && dev < 64 && cache[dev]) return cache[dev];
  void* p = nullptr;
  *err = cudaGetSymbolAddress(&p, g_static_scratch);
  if (*err != cudaSuccess) return nullptr;
  if (dev >= 0 && dev < 64) cache[dev] = p;
  return p;
}

}  // namespace

extern "C" {

int mx_quantize_host_static(const void* in_host, void* elems_out_host, uint8_t* scales_out_host,
                            const int64_t* shape, int ndim, int axis, mx_fmt_t fmt,
                            mx_round_t rounding, const mx_opts_t* opts) {
  // size check first: an oversized request is refused before anything touches the device
  Opts o;
  View v;
  if (!shape) return MX_ERR_NULL;
  if (!fmt_ok((int)fmt) || !read_opts(opts, &o)) return MX_ERR_FMT;
  if (o.pad128) return MX_ERR_UNSUPPORTED;  // zero-extended rows: mx_quantize and mx_gemm* only
  if (!make_view(shape, ndim, axis, &v)) return MX_ERR_SHAPE;
  if (mx_quantize_host_workspace_bytes(shape, ndim, axis, fmt, opts) > MX_STATIC_SCRATCH_BYTES)
    return MX_ERR_WORKSPACE;
  cudaError_t e;
  void* scratch = static_scratch_address(&e);
  if (!scratch) return fail_cuda(e);
  // mx_quantize_host copies the input in, zeroes the scale padding where there is any, runs
  // the kernel and copies exactly the produced bytes out: nothing stale is ever read back.
  return quantize_host_impl(in_host, elems_out_host, scales_out_host, shape, ndim, axis, fmt, rounding, opts,
                            scratch, MX_STATIC_SCRATCH_BYTES, false);  // one stream, nothing created
}

size_t mx_dequantize_host_workspace_bytes(const int64_t* shape, int ndim, int axis, mx_fmt_t fmt,
                                          const mx_opts_t* opts) {
  return mx_quantize_host_workspace_bytes(shape, ndim, axis, fmt, opts);
}

static int dequantize_host_impl(const void* elems_host, const uint8_t* scales_host, void* out_host,
                                const int64_t* shape, int ndim, int axis, mx_fmt_t fmt, const mx_opts_t* opts,
                                void* workspace_dev, size_t workspace_bytes, bool async) {
  Opts o;
  View v;
  if (!shape) return MX_ERR_NULL;
  if (!fmt_ok((int)fmt) || !read_opts(opts, &o)) return MX_ERR_FMT;
  if (o.pad128) return MX_ERR_UNSUPPORTED;  // zero-extended rows: mx_quantize and mx_gemm* only
  if (!make_view(shape, ndim, axis, &v)) return MX_ERR_SHAPE;
  if (axis != ndim - 1) return MX_ERR_UNSUPPORTED;
  if (v.numel == 0) return MX_OK;
  if (!elems_host || !scales_host || !out_host || !workspace_dev) return MX_ERR_NULL;
  if ((uintptr_t)workspace_dev % 256) return MX_ERR_ALIGN;
  if (workspace_bytes < mx_dequantize_host_workspace_bytes(shape, ndim, axis, fmt, opts))
    return MX_ERR_WORKSPACE;
  const size_t out_b = (size_t)v.numel * (o.dtype == MX_BF16 ? 2 : 4);
  const size_t el_b = (size_t)v.padded_numel / 8 * fmt_bits((int)fmt);
  const size_t sc_b = scales_bytes(v.rows, v.kblocks, o.layout);
  char* d_out = (char*)workspace_dev;
  char* d_el = d_out + align_up(out_b, 256);
  char* d_sc = d_el + align_up(el_b, 256);
  cudaError_t e;
  int64_t rpc = v.rows;
  const int chunks = plan_chunks(v.rows, out_b, &rpc);
  if (chunks > 1 || async) {  // row chunks over two streams, as in quantize_host_impl
    HostPipe* hp = host_pipe(&e);
    if (!hp) return fail_cuda(e);
    if ((e = cudaEventRecord(hp->start, o.stream)) != cudaSuccess ||
        (e = cudaStreamWaitEvent(hp->in, hp->start, 0)) != cudaSuccess ||
        (e = cudaStreamWaitEvent(hp->out, hp->start, 0)) != cudaSuccess)
      return fail_cuda(e);
    mx_opts_t co = {o.dtype, o.layout, hp->in, 0};
    const size_t row_out = (size_t)v.L * (o.dtype == MX_BF16 ? 2 : 4), row_el = (size_t)v.Lp / 8 * fmt_bits((int)fmt);
    for (int c = 0; c < chunks; ++c) {
      const int64_t r0 = c * rpc, nr = (r0 + rpc <= v.rows ? rpc : v.rows - r0);
      const size_t so = scales_row_offset(r0, v.kblocks, o.layout);
      const size_t sb = scales_bytes(nr, v.kblocks, o.layout);
      if (c == 0 && (e = cudaMemcpyAsync(d_sc, scales_host, sc_b, cudaMemcpyHostToDevice, hp->in)) != cudaSuccess)
        return fail_cuda(e);  // the whole (small) scale tensor goes first
      (void)sb;
      if ((e = cudaMemcpyAsync(d_el + r0 * row_el, (const char*)elems_host + r0 * row_el, nr * row_el,
                               cudaMemcpyHostToDevice, hp->in)) != cudaSuccess)
        return fail_cuda(e);
      const int64_t cshape[2] = {nr, v.L};
      const int rc = mx_dequantize(d_el + r0 * row_el, (const uint8_t*)d_sc + so, d_out + r0 * row_out, cshape, 2, 1,
                                   fmt, &co);
      if (rc != MX_OK) return rc;
      if ((e = cudaEventRecord(hp->done[c], hp->in)) != cudaSuccess ||
          (e = cudaStreamWaitEvent(hp->out, hp->done[c], 0)) != cudaSuccess ||
          (e = cudaMemcpyAsync((char*)out_host + r0 * row_out, d_out + r0 * row_out, nr * row_out,
                               cudaMemcpyDeviceToHost, hp->out)) != cudaSuccess)
        return fail_cuda(e);
    }
    if (async) return MX_OK;
    if ((e = cudaStreamSynchronize(hp->out)) != cudaSuccess || (e = cudaStreamSynchronize(hp->in)) != cudaSuccess ||
        (e = cudaStreamSynchronize(o.stream)) != cudaSuccess)
      return fail_cuda(e);
    return MX_OK;
  }
  e = cudaMemcpyAsync(d_el, elems_host, el_b, cudaMemcpyHostToDevice, o.stream);
  if (e != cudaSuccess) return fail_cuda(e);
  e = cudaMemcpyAsync(d_sc, scales_host, sc_b, cudaMemcpyHostToDevice, o.stream);
  if (e != cudaSuccess) return fail_cuda(e);
  const int rc = mx_dequantize(d_el, (const uint8_t*)d_sc, d_out, shape, ndim, axis, fmt, opts);
  if (rc != MX_OK) return rc;
  e = cudaMemcpyAsync(out_host, d_out, out_b, cudaMemcpyDeviceToHost, o.stream);
  if (e != cudaSuccess) return fail_cuda(e);
  e = cudaStreamSynchronize(o.stream);
  return e == cudaSuccess ? MX_OK : fail_cuda(e);
}

int mx_dequantize_host(const void* elems_host, const uint8_t* scales_host, void* out_host,
                       const int64_t* shape, int ndim, int axis, mx_fmt_t fmt,
                       const mx_opts_t* opts, void* workspace_dev, size_t workspace_bytes) {
  return dequantize_host_impl(elems_host, scales_host, out_host, shape, ndim, axis, fmt, opts, workspace_dev,
                              workspace_bytes, false);
}

int mx_quantize_host_async(const void* in_host, void* elems_out_host, uint8_t* scales_out_host,
                           const int64_t* shape, int ndim, int axis, mx_fmt_t fmt, mx_round_t rounding,
                           const mx_opts_t* opts, void* workspace_dev, size_t workspace_bytes) {
  return quantize_host_impl(in_host, elems_out_host, scales_out_host, shape, ndim, axis, fmt, rounding, opts,
                            workspace_dev, workspace_bytes, true, true);
}

int mx_dequantize_host_async(const void* elems_host, const uint8_t* scales_host, void* out_host,
                             const int64_t* shape, int ndim, int axis, mx_fmt_t fmt,
                             const mx_opts_t* opts, void* workspace_dev, size_t workspace_bytes) {
  return dequantize_host_impl(elems_host, scales_host, out_host, shape, ndim, axis, fmt, opts, workspace_dev,
                              workspace_bytes, true);
}

int mx_host_synchronize(void) {
  cudaError_t e;
  HostPipe* hp = host_pipe(&e);
  if (!hp) return fail_cuda(e);
  if ((e = cudaStreamSynchronize(hp->in)) != cudaSuccess || (e = cudaStreamSynchronize(hp->out)) != cudaSuccess)
    return fail_cuda(e);
  return MX_OK;
}

// ---------------------------------------------------------------------------
// GEMM
// ---------------------------------------------------------------------------

constexpr int kFewRowsDefault = 96;  // largest M that takes the swapped-operand kernel

// strict: every matrix must consist of whole 128-row / 128-column tiles (batched products, whose
// matrices are stacked along rows, and the quantizing epilogue, which writes whole blocks).
static int gemm_validate(const void* A, const uint8_t* sA, const void* B, const uint8_t* sB,
                         const void* C, int64_t M, int64_t N, int64_t K, int fmtA, int fmtB,
                         bool strict, int c_elem_bytes) {
  if (!A || !sA || !B || !sB || !C) return MX_ERR_NULL;
  if (!fmt_ok(fmtA) || !fmt_ok(fmtB)) return MX_ERR_FMT;
  if (fmtA == MX_INT8 || fmtB == MX_INT8) return MX_ERR_UNSUPPORTED;
  if (M < 0 || N < 0 || K < 32 || K % 32) return MX_ERR_SHAPE;
  // the tensor-map types of packed 6- and 4-bit codes take rows of whole 128-element groups only
  if ((fmt_bits(fmtA) < 8 || fmt_bits(fmtB) < 8) && K % 128) return MX_ERR_SHAPE;
  if (strict ? (M % 128 || N % 128) : (N * c_elem_bytes) % 16 != 0) return MX_ERR_SHAPE;
  if (M >= ((int64_t)1 << 31) || N >= ((int64_t)1 << 31) || K >= ((int64_t)1 << 31)) return MX_ERR_SHAPE;
  return MX_OK;
}

// C != NULL: scalar-float output; otherwise q_elems / q_scales receive C as an MX tensor.
static int gemm_device(const void* A, const uint8_t* sA, const void* B, const uint8_t* sB, void* C,
                       int c_bf16, int64_t batch, int64_t M, int64_t N, int64_t K, mx_fmt_t fmtA,
                       mx_fmt_t fmtB, const mx_opts_t* opts, void* q_elems = nullptr,
                       uint8_t* q_scales = nullptr, int q_fmt = 0, int q_round = 0,
                       const mx_gemm_plan_t* plan = nullptr) {
  Opts o;
  if (!C) {
    if (!q_elems || !q_scales) return MX_ERR_NULL;
    C = q_elems;  // stands in for the output pointer in the checks below
  }
  if (!read_opts(opts, &o)) return MX_ERR_FMT;
  if (o.pad128) {
    // Operands stored as the tensors zero-extended along K to a multiple of 128 (mx_quantize with
    // the same option): the product over the extended K is the product over K, term for term.
    if (batch != 1 || q_elems != nullptr) return MX_ERR_UNSUPPORTED;
    if (K < 32 || K % 32 || K >= ((int64_t)1 << 31) - 128) return MX_ERR_SHAPE;
    K = (K + 127) / 128 * 128;
  }
  int rc = gemm_validate(A, sA, B, sB, C, M, N, K, (int)fmtA, (int)fmtB, batch != 1 || q_elems != nullptr,
                         c_bf16 ? 2 : 4);
  if (rc != MX_OK) return rc;
  if (o.layout != MX_SCALES_SWIZZLED) return MX_ERR_UNSUPPORTED;
  if ((uintptr_t)A % 32 || (uintptr_t)B % 32 || (uintptr_t)sA % 16 || (uintptr_t)sB % 16 ||
      (uintptr_t)C % 16)
    return MX_ERR_ALIGN;
  if (batch < 0 || batch * M >= ((int64_t)1 << 31) || batch * N >= ((int64_t)1 << 31) ||
      (M > 0 && N > 0 && batch * ((M + 127) / 128) * ((N + 127) / 128) >= ((int64_t)1 << 31)))
    return MX_ERR_SHAPE;
  if (M == 0 || N == 0 || batch == 0) return MX_OK;
  cudaError_t e;
  mx::GemmArgs a;
  a.A = A; a.sA = sA; a.B = B; a.sB = sB; a.C = C; a.c_bf16 = c_bf16; a.batch = batch;
  a.dense = 0;
  a.force_bn = plan ? plan->tile_n : 0;
  a.skinny_m = plan && plan->few_rows_limit >= 0 ? plan->few_rows_limit : kFewRowsDefault;
  a.wait_cycles = plan ? plan->wait_cycles : 0;
  a.drop_fill = plan ? plan->drop_fill : -1;
  a.q_elems = q_elems; a.q_scales = q_scales; a.q_fmt = q_fmt; a.q_round = q_round;
  a.M = M; a.N = N; a.K = K; a.fmtA = (int)fmtA; a.fmtB = (int)fmtB;
  a.stream = o.stream;
  a.sm_count = sm_count(&e);
  if (e != cudaSuccess) return fail_cuda(e);
  rc = mx::launch_gemm(a, &e);
  if (rc != MX_OK) return rc == MX_ERR_CUDA ? fail_cuda(e) : rc;
  if (o.check) {
    unsigned int st = 0;
    rc = mx::gemm_status(o.stream, &st, &e);
    if (rc != MX_OK) return fail_cuda(e);
    if (st != 0) {
      std::snprintf(g_cuda_error, sizeof(g_cuda_error), "device-side wait %u gave up "
                    "(1 producer/stage empty, 2 MMA/stage full, 3 MMA/accumulator free, "
                    "4 epilogue/accumulator full, 5 scale copier/stage full, 6 shared-memory alignment)", st);
      return MX_ERR_TIMEOUT;
    }
  }
  return MX_OK;
}

int mx_gemm(const void* A, const uint8_t* sA, const void* B, const uint8_t* sB, float* C,
            int64_t M, int64_t N, int64_t K, mx_fmt_t fmtA, mx_fmt_t fmtB, const mx_opts_t* opts) {
  return gemm_device(A, sA, B, sB, C, 0, 1, M, N, K, fmtA, fmtB, opts);
}

int mx_gemm_bf16(const void* A, const uint8_t* sA, const void* B, const uint8_t* sB, void* C,
                 int64_t M, int64_t N, int64_t K, mx_fmt_t fmtA, mx_fmt_t fmtB,
                 const mx_opts_t* opts) {
  return gemm_device(A, sA, B, sB, C, 1, 1, M, N, K, fmtA, fmtB, opts);
}

int mx_gemm_ex(const void* A, const uint8_t* sA, const void* B, const uint8_t* sB, void* C,
               int64_t M, int64_t N, int64_t K, mx_fmt_t fmtA, mx_fmt_t fmtB,
               const mx_opts_t* opts, const mx_gemm_plan_t* plan) {
  if (!plan) return gemm_device(A, sA, B, sB, C, 0, 1, M, N, K, fmtA, fmtB, opts);
  if (plan->c_dtype != MX_F32 && plan->c_dtype != MX_BF16) return MX_ERR_FMT;
  if ((plan->tile_n != 0 && plan->tile_n != 256 && plan->tile_n != 384) || plan->few_rows_limit < -1 ||
      plan->few_rows_limit > 128 || plan->drop_fill < -1 || plan->wait_cycles < 0)
    return MX_ERR_SHAPE;
  return gemm_device(A, sA, B, sB, C, plan->c_dtype == MX_BF16, 1, M, N, K, fmtA, fmtB, opts, nullptr, nullptr,
                     0, 0, plan);
}

int mx_gemm_batched(const void* A, const uint8_t* sA, const void* B, const uint8_t* sB, void* C,
                    mx_dtype_t c_dtype, int64_t batch, int64_t M, int64_t N, int64_t K,
                    mx_fmt_t fmtA, mx_fmt_t fmtB, const mx_opts_t* opts) {
  if ((int)c_dtype != MX_F32 && (int)c_dtype != MX_BF16) return MX_ERR_FMT;
  return gemm_device(A, sA, B, sB, C, (int)c_dtype == MX_BF16, batch, M, N, K, fmtA, fmtB, opts);
}

int mx_gemm_quantize(const void* A, const uint8_t* sA, const void* B, const uint8_t* sB,
                     void* elems_out, uint8_t* scales_out, int64_t M, int64_t N, int64_t K,
                     mx_fmt_t fmtA, mx_fmt_t fmtB, mx_fmt_t fmtC, mx_round_t rounding,
                     const mx_opts_t* opts) {
  if (!elems_out || !scales_out) return MX_ERR_NULL;
  if (!fmt_ok((int)fmtC) || ((int)rounding != MX_RNE && (int)rounding != MX_RHAZ)) return MX_ERR_FMT;
  if ((uintptr_t)scales_out % 16) return MX_ERR_ALIGN;
  return gemm_device(A, sA, B, sB, nullptr, 0, 1, M, N, K, fmtA, fmtB, opts, elems_out, scales_out,
                     (int)fmtC, (int)rounding);
}

size_t mx_gemm_dense_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  if (M < 0 || N < 0 || K < 0) return 0;
  return align_up((size_t)M * (size_t)K * 2, 256) + align_up((size_t)N * (size_t)K * 2, 256);
}

int mx_gemm_dense(const void* A, const uint8_t* sA, const void* B, const uint8_t* sB, void* C,
                  mx_dtype_t c_dtype, int64_t M, int64_t N, int64_t K, mx_fmt_t fmtA, mx_fmt_t fmtB,
                  const mx_opts_t* opts, void* workspace, size_t workspace_bytes) {
  Opts o;
  if (!A || !sA || !B || !sB || !C) return MX_ERR_NULL;
  if (!fmt_ok((int)fmtA) || !fmt_ok((int)fmtB) || !read_opts(opts, &o)) return MX_ERR_FMT;
  if (o.pad128) return MX_ERR_UNSUPPORTED;  // zero-extended rows: mx_quantize and mx_gemm* only
  if ((int)c_dtype != MX_F32 && (int)c_dtype != MX_BF16) return MX_ERR_FMT;
  if (M < 0 || N < 0 || K < 32 || K % 32 || (N * ((int)c_dtype == MX_BF16 ? 2 : 4)) % 16) return MX_ERR_SHAPE;
  if (M >= ((int64_t)1 << 31) || N >= ((int64_t)1 << 31) || K >= ((int64_t)1 << 31)) return MX_ERR_SHAPE;
  if (o.layout != MX_SCALES_SWIZZLED) return MX_ERR_UNSUPPORTED;
  if ((uintptr_t)A % 16 || (uintptr_t)B % 16 || (uintptr_t)sA % 16 || (uintptr_t)sB % 16 ||
      (uintptr_t)C % 16)
    return MX_ERR_ALIGN;
  if (M == 0 || N == 0) return MX_OK;
  if (!workspace) return MX_ERR_NULL;
  if ((uintptr_t)workspace % 256) return MX_ERR_ALIGN;
  if (workspace_bytes < mx_gemm_dense_workspace_bytes(M, N, K)) return MX_ERR_WORKSPACE;
  if (M * K / 8 >= (int64_t)1 << 31 || N * K / 8 >= (int64_t)1 << 31) return MX_ERR_UNSUPPORTED;
  char* dA = (char*)workspace;
  char* dB = dA + align_up((size_t)M * (size_t)K * 2, 256);
  cudaError_t e;
  const int sms = sm_count(&e);
  if (e != cudaSuccess) return fail_cuda(e);
  mx::DequantizeArgs d;
  d.dtype = MX_BF16; d.layout = MX_SCALES_SWIZZLED; d.stream = o.stream; d.sm_count = sms;
  d.elems = (const uint8_t*)A; d.scales = sA; d.out = dA; d.rows = M; d.L = K; d.fmt = (int)fmtA;
  if ((e = mx::launch_dequantize(d)) != cudaSuccess) return fail_cuda(e);
  d.elems = (const uint8_t*)B; d.scales = sB; d.out = dB; d.rows = N; d.L = K; d.fmt = (int)fmtB;
  if ((e = mx::launch_dequantize(d)) != cudaSuccess) return fail_cuda(e);
  mx::GemmArgs a;
  a.A = dA; a.sA = nullptr; a.B = dB; a.sB = nullptr; a.C = C; a.c_bf16 = (int)c_dtype == MX_BF16;
  a.dense = 1; a.batch = 1; a.force_bn = 0; a.skinny_m = 0; a.wait_cycles = 0; a.drop_fill = -1;
  a.q_elems = nullptr; a.q_scales = nullptr; a.q_fmt = 0; a.q_round = 0;
  a.M = M; a.N = N; a.K = K; a.fmtA = (int)fmtA; a.fmtB = (int)fmtB;
  a.stream = o.stream; a.sm_count = sms;
  int rc = mx::launch_gemm(a, &e);
  if (rc != MX_OK) return rc == MX_ERR_CUDA ? fail_cuda(e) : rc;
  if (o.check) {
    unsigned int st = 0;
    rc = mx::gemm_status(o.stream, &st, &e);
    if (rc != MX_OK) return fail_cuda(e);
    if (st != 0) {
      std::snprintf(g_cuda_error, sizeof(g_cuda_error), "device-side wait %u gave up "
                    "(1 producer/stage empty, 2 MMA/stage full, 3 MMA/accumulator free, "
                    "4 epilogue/accumulator full, 5 scale copier/stage full, 6 shared-memory alignment)", st);
      return MX_ERR_TIMEOUT;
    }
  }
  return MX_OK;
}

static bool conv_ok(const mx_conv_t* c) {
  return c && c->N >= 0 && c->H > 0 && c->W > 0 && c->C > 0 && c->kh > 0 && c->kw > 0 && c->stride_h > 0 &&
         c->stride_w > 0 && c->pad_h >= 0 && c->pad_w >= 0 && c->dil_h > 0 && c->dil_w > 0 &&
         c->H < ((int64_t)1 << 30) && c->W < ((int64_t)1 << 30);
}

int64_t mx_conv_out_h(const mx_conv_t* c) {
  if (!conv_ok(c)) return 0;
  const int64_t span = c->H + 2 * (int64_t)c->pad_h - (int64_t)c->dil_h * (c->kh - 1) - 1;
  return span < 0 ? 0 : span / c->stride_h + 1;
}

int64_t mx_conv_out_w(const mx_conv_t* c) {
  if (!conv_ok(c)) return 0;
  const int64_t span = c->W + 2 * (int64_t)c->pad_w - (int64_t)c->dil_w * (c->kw - 1) - 1;
  return span < 0 ? 0 : span / c->stride_w + 1;
}

int mx_im2col(const void* elems_in, const uint8_t* scales_in, void* elems_out, uint8_t* scales_out,
              const mx_conv_t* conv, mx_fmt_t fmt, const mx_opts_t* opts) {
  Opts o;
  if (!conv) return MX_ERR_NULL;
  if (!fmt_ok((int)fmt) || !read_opts(opts, &o)) return MX_ERR_FMT;
  if (o.pad128) return MX_ERR_UNSUPPORTED;  // zero-extended rows: mx_quantize and mx_gemm* only
  if (!conv_ok(conv)) return MX_ERR_SHAPE;
  const int bits = fmt_bits((int)fmt);
  if (conv->C % 32 || (conv->C * bits / 8) % 16) return MX_ERR_SHAPE;
  const int64_t Ho = mx_conv_out_h(conv), Wo = mx_conv_out_w(conv);
  if (Ho <= 0 || Wo <= 0) return MX_ERR_SHAPE;
  const int64_t taps = (int64_t)conv->kh * conv->kw;
  const int64_t M = conv->N * Ho * Wo;
  // 32-bit chunk indices in the gather: the output holds fewer than 2^32 16-byte chunks
  if (conv->N * conv->H * conv->W >= ((int64_t)1 << 31) || M * taps * (conv->C * bits / 8 / 16) >= ((int64_t)1 << 32) ||
      M * taps >= ((int64_t)1 << 31) || taps * conv->C >= ((int64_t)1 << 31))
    return MX_ERR_SHAPE;
  if (M == 0) return MX_OK;
  if (!elems_in || !scales_in || !elems_out || !scales_out) return MX_ERR_NULL;
  if ((uintptr_t)elems_in % 16 || (uintptr_t)scales_in % 16 || (uintptr_t)elems_out % 16 ||
      (uintptr_t)scales_out % 16)
    return MX_ERR_ALIGN;
  cudaError_t e;
  mx::Im2colArgs a;
  a.elems_in = (const uint8_t*)elems_in; a.scales_in = scales_in;
  a.elems_out = (uint8_t*)elems_out; a.scales_out = scales_out;
  a.N = conv->N; a.H = conv->H; a.W = conv->W; a.C = conv->C; a.Ho = Ho; a.Wo = Wo;
  a.kh = conv->kh; a.kw = conv->kw; a.stride_h = conv->stride_h; a.stride_w = conv->stride_w;
  a.pad_h = conv->pad_h; a.pad_w = conv->pad_w; a.dil_h = conv->dil_h; a.dil_w = conv->dil_w;
  a.bits = bits; a.layout_in = o.layout; a.stream = o.stream;
  a.sm_count = sm_count(&e);
  if (e != cudaSuccess) return fail_cuda(e);
  e = mx::launch_im2col(a);
  return e == cudaSuccess ? MX_OK : fail_cuda(e);
}

int mx_conv2d(const void* x_elems, const uint8_t* x_scales, const void* w_elems, const uint8_t* w_scales,
              void* y, mx_dtype_t y_dtype, const mx_conv_t* conv, int64_t Cout, mx_fmt_t fmt_x,
              mx_fmt_t fmt_w, const mx_opts_t* opts) {
  Opts o;
  if (!conv) return MX_ERR_NULL;
  if (!fmt_ok((int)fmt_x) || !fmt_ok((int)fmt_w) || !read_opts(opts, &o)) return MX_ERR_FMT;
  if (o.pad128) return MX_ERR_UNSUPPORTED;  // zero-extended rows: mx_quantize and mx_gemm* only
  if ((int)y_dtype != MX_F32 && (int)y_dtype != MX_BF16) return MX_ERR_FMT;
  if (!conv_ok(conv)) return MX_ERR_SHAPE;
  if (fmt_x == MX_INT8 || fmt_w == MX_INT8 || fmt_bits((int)fmt_x) != 8) return MX_ERR_UNSUPPORTED;
  const int64_t Ho = mx_conv_out_h(conv), Wo = mx_conv_out_w(conv);
  const int64_t K = (int64_t)conv->kh * conv->kw * conv->C;
  const int esz = (int)y_dtype == MX_BF16 ? 2 : 4;
  if (Ho <= 0 || Wo <= 0 || conv->C % 32 || Cout < 0 || (Cout * esz) % 16) return MX_ERR_SHAPE;
  if (fmt_bits((int)fmt_w) < 8 && K % 128) return MX_ERR_SHAPE;
  const int64_t M = conv->N * Ho * Wo;
  if (M >= ((int64_t)1 << 31) || Cout >= ((int64_t)1 << 31) || K >= ((int64_t)1 << 31) ||
      conv->N * conv->H * conv->W >= ((int64_t)1 << 31) ||
      (M > 0 && Cout > 0 && ((M + 127) / 128) * ((Cout + 127) / 128) >= ((int64_t)1 << 31)))
    return MX_ERR_SHAPE;
  if (M == 0 || Cout == 0) return MX_OK;
  if (!x_elems || !x_scales || !w_elems || !w_scales || !y) return MX_ERR_NULL;
  if ((uintptr_t)x_elems % 16 || (uintptr_t)x_scales % 16 || (uintptr_t)w_elems % 32 || (uintptr_t)w_scales % 16 ||
      (uintptr_t)y % 16)
    return MX_ERR_ALIGN;
  cudaError_t e;
  mx::ConvArgs a;
  a.x_elems = (const uint8_t*)x_elems; a.x_scales = x_scales; a.w_elems = w_elems; a.w_scales = w_scales;
  a.y = y; a.y_bf16 = (int)y_dtype == MX_BF16;
  a.N = conv->N; a.H = conv->H; a.W = conv->W; a.C = conv->C; a.Ho = Ho; a.Wo = Wo; a.Cout = Cout;
  a.kh = conv->kh; a.kw = conv->kw; a.stride_h = conv->stride_h; a.stride_w = conv->stride_w;
  a.pad_h = conv->pad_h; a.pad_w = conv->pad_w; a.dil_h = conv->dil_h; a.dil_w = conv->dil_w;
  a.fmt_x = (int)fmt_x; a.fmt_w = (int)fmt_w; a.x_layout = o.layout; a.stream = o.stream;
  a.sm_count = sm_count(&e);
  if (e != cudaSuccess) return fail_cuda(e);
  int rc = mx::launch_conv(a, &e);
  if (rc != MX_OK) return rc == MX_ERR_CUDA ? fail_cuda(e) : rc;
  if (o.check) {
    unsigned int st = 0;
    rc = mx::gemm_status(o.stream, &st, &e);
    if (rc != MX_OK) return fail_cuda(e);
    if (st != 0) {
      std::snprintf(g_cuda_error, sizeof(g_cuda_error), "device-side wait %u gave up "
                    "(1 producer/stage empty, 2 MMA/stage full, 3 MMA/accumulator free, "
                    "4 epilogue/accumulator full, 5 scale copier/stage full, 6 shared-memory alignment)", st);
      return MX_ERR_TIMEOUT;
    }
  }
  return MX_OK;
}

size_t mx_gemm_host_workspace_bytes(int64_t M, int64_t N, int64_t K, mx_fmt_t fmtA, mx_fmt_t fmtB) {
  if (!fmt_ok((int)fmtA) || !fmt_ok((int)fmtB) || M < 0 || N < 0 || K < 0 || K % 32) return 0;
  return align_up((size_t)(M * K / 8 * fmt_bits((int)fmtA)), 256) +
         align_up(scales_bytes(M, K / 32, MX_SCALES_SWIZZLED), 256) +
         align_up((size_t)(N * K / 8 * fmt_bits((int)fmtB)), 256) +
         align_up(scales_bytes(N, K / 32, MX_SCALES_SWIZZLED), 256) +
         align_up((size_t)(M * N) * 4, 256);
}

int mx_gemm_host(const void* A_host, const uint8_t* sA_host, const void* B_host,
                 const uint8_t* sB_host, float* C_host, int64_t M, int64_t N, int64_t K,
                 mx_fmt_t fmtA, mx_fmt_t fmtB, const mx_opts_t* opts, void* workspace_dev,
                 size_t workspace_bytes) {
  Opts o;
  int rc = gemm_validate(A_host, sA_host, B_host, sB_host, C_host, M, N, K, (int)fmtA, (int)fmtB, false, 4);
  if (rc != MX_OK) return rc;
  if (!read_opts(opts, &o)) return MX_ERR_FMT;
  if (o.pad128) return MX_ERR_UNSUPPORTED;  // zero-extended rows: mx_quantize and mx_gemm* only
  if (!workspace_dev) return MX_ERR_NULL;
  if ((uintptr_t)workspace_dev % 256) return MX_ERR_ALIGN;
  if (workspace_bytes < mx_gemm_host_workspace_bytes(M, N, K, fmtA, fmtB)) return MX_ERR_WORKSPACE;
  if (M == 0 || N == 0) return MX_OK;
  const size_t a_b = (size_t)(M * K / 8 * fmt_bits((int)fmtA));
  const size_t sa_b = scales_bytes(M, K / 32, MX_SCALES_SWIZZLED);
  const size_t b_b = (size_t)(N * K / 8 * fmt_bits((int)fmtB));
  const size_t sb_b = scales_bytes(N, K / 32, MX_SCALES_SWIZZLED);
  const size_t c_b = (size_t)(M * N) * 4;
  char* dA = (char*)workspace_dev;
  char* dsA = dA + align_up(a_b, 256);
  char* dB = dsA + align_up(sa_b, 256);
  char* dsB = dB + align_up(b_b, 256);
  char* dC = dsB + align_up(sb_b, 256);
  cudaError_t e;
  if ((e = cudaMemcpyAsync(dA, A_host, a_b, cudaMemcpyHostToDevice, o.stream)) != cudaSuccess ||
      (e = cudaMemcpyAsync(dsA, sA_host, sa_b, cudaMemcpyHostToDevice, o.stream)) != cudaSuccess ||
      (e = cudaMemcpyAsync(dB, B_host, b_b, cudaMemcpyHostToDevice, o.stream)) != cudaSuccess ||
      (e = cudaMemcpyAsync(dsB, sB_host, sb_b, cudaMemcpyHostToDevice, o.stream)) != cudaSuccess)
    return fail_cuda(e);
  rc = mx_gemm(dA, (const uint8_t*)dsA, dB, (const uint8_t*)dsB, (float*)dC, M, N, K, fmtA, fmtB, opts);
  if (rc != MX_OK) return rc;
  if ((e = cudaMemcpyAsync(C_host, dC, c_b, cudaMemcpyDeviceToHost, o.stream)) != cudaSuccess)
    return fail_cuda(e);
  e = cudaStreamSynchronize(o.stream);
  return e == cudaSuccess ? MX_OK : fail_cuda(e);
}

}  // extern "C"
