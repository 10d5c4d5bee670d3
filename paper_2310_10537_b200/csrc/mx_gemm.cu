// placeholder: block-scaled GEMM (filled in next)
#include "mx.h"
#include "mx_launch.h"
extern "C" {
int mx_gemm(const void*, const uint8_t*, const void*, const uint8_t*, float*, int64_t, int64_t,
            int64_t, mx_fmt_t, mx_fmt_t, const mx_opts_t*) { return MX_ERR_UNSUPPORTED; }
size_t mx_gemm_host_workspace_bytes(int64_t, int64_t, int64_t, mx_fmt_t, mx_fmt_t) { return 0; }
int mx_gemm_host(const void*, const uint8_t*, const void*, const uint8_t*, float*, int64_t,
                 int64_t, int64_t, mx_fmt_t, mx_fmt_t, const mx_opts_t*, void*, size_t) {
  return MX_ERR_UNSUPPORTED;
}
}
