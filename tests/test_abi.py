"""CPU-only checks of the C ABI: the library loads, exports every symbol the
public header declares, its size / index helpers agree with the oracle's own
restatement of the layouts, and argument validation returns the documented
status codes without touching a GPU."""
import ctypes
import os
import re

import numpy as np

import oracle as O
import paper_2310_10537_b200 as mx

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "mx.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mx_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_functions()
    assert "mx_quantize" in names and "mx_gemm" in names and len(names) >= 15
    lib = ctypes.CDLL(mx.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(mx.EXPORTS) == names


def test_helpers_match_oracle_layouts():
    for fmt in range(6):
        assert mx.mx_fmt_bits(fmt) == O.fmt_bits(fmt)
        assert mx.mx_elems_bytes([3, 64, 5], 1, fmt) == 3 * 64 * 5 * O.fmt_bits(fmt) // 8
    assert mx.mx_fmt_bits(6) == 0
    for rows, kb in ((1, 1), (128, 4), (200, 7), (257, 9)):
        for layout in (0, 1):
            assert mx.mx_scales_bytes([rows, kb * 32], 1, layout) == O.scales_bytes(rows, kb, layout)
            for r in range(0, rows, 13):
                for k in range(kb):
                    assert mx.mx_scale_offset(r, k, rows, kb, layout) == O.scale_offset(r, k, rows, kb, layout)
    assert mx.mx_scale_offset(5, 0, 5, 1, 1) == ctypes.c_size_t(-1).value
    assert mx.mx_elems_bytes([4, 33], 1, 0) == 4 * 64          # a partial block is stored padded
    assert mx.mx_scales_bytes([4, 33], 1, 0) == 4 * 2
    assert mx.mx_scales_bytes([4, 64], 2, 0) == 0


def test_argument_validation_without_gpu():
    lib = mx.lib()
    shape = (ctypes.c_int64 * 2)(4, 64)
    buf = np.zeros(4096, np.uint8)
    p = buf.ctypes.data + (-buf.ctypes.data) % 64
    o = mx.binding.mx_opts_t(mx.MX_F32, mx.MX_SCALES_LINEAR, None, 0)
    q = lib.mx_quantize
    assert q(None, p, p, shape, 2, 1, 0, 0, ctypes.byref(o)) == mx.MX_ERR_NULL
    assert q(p, p, p, None, 2, 1, 0, 0, ctypes.byref(o)) == mx.MX_ERR_NULL
    assert q(p, p, p, shape, 2, 2, 0, 0, ctypes.byref(o)) == mx.MX_ERR_SHAPE
    assert q(p, p, p, shape, 0, 0, 0, 0, ctypes.byref(o)) == mx.MX_ERR_SHAPE
    assert q(p, p, p, shape, 2, 1, 6, 0, ctypes.byref(o)) == mx.MX_ERR_FMT
    assert q(p, p, p, shape, 2, 1, 0, 2, ctypes.byref(o)) == mx.MX_ERR_FMT
    assert q(p + 4, p, p, shape, 2, 1, 0, 0, ctypes.byref(o)) == mx.MX_ERR_ALIGN
    bad = mx.binding.mx_opts_t(7, 0, None, 0)
    assert q(p, p, p, shape, 2, 1, 0, 0, ctypes.byref(bad)) == mx.MX_ERR_FMT
    empty = (ctypes.c_int64 * 2)(0, 64)
    assert q(None, None, None, empty, 2, 1, 0, 0, ctypes.byref(o)) == mx.MX_OK
    d = lib.mx_dequantize
    assert d(p, p, p, shape, 2, 0, 0, ctypes.byref(o)) == mx.MX_ERR_UNSUPPORTED   # blocks must run along the last axis
    neg = (ctypes.c_int64 * 2)(4, -64)
    assert d(p, p, p, neg, 2, 1, 0, ctypes.byref(o)) == mx.MX_ERR_SHAPE
    assert q(p, p, p, neg, 2, 1, 0, 0, ctypes.byref(o)) == mx.MX_ERR_SHAPE
    shape3 = (ctypes.c_int64 * 2)(64, 4)
    assert d(p, p, p, shape3, 2, 0, 0, ctypes.byref(o)) == mx.MX_ERR_UNSUPPORTED
    assert d(p, None, p, shape, 2, 1, 0, ctypes.byref(o)) == mx.MX_ERR_NULL
    g = lib.mx_gemm
    assert g(p, p, p, p, p, -1, 128, 128, 0, 0, None) == mx.MX_ERR_SHAPE
    assert g(p, p, p, p, p, 128, 130, 128, 0, 0, None) == mx.MX_ERR_SHAPE   # C rows not whole 16-byte units
    assert g(p, p, p, p, p, 128, 128, 48, 0, 0, None) == mx.MX_ERR_SHAPE    # K not a multiple of 32
    assert g(p, p, p, p, p, 128, 128, 96, 2, 0, None) == mx.MX_ERR_SHAPE    # 6- and 4-bit codes need K % 128
    assert g(p, p, p, p, p, 128, 128, 128, 5, 0, None) == mx.MX_ERR_UNSUPPORTED
    assert g(p, p, p, p, p, 128, 128, 128, 0, 9, None) == mx.MX_ERR_FMT
    assert g(None, p, p, p, p, 128, 128, 128, 0, 0, None) == mx.MX_ERR_NULL
    assert lib.mx_strerror(mx.MX_ERR_ALIGN) and lib.mx_strerror(-99)


def test_pad_k128_option_is_validated_without_gpu():
    """pad_k128 takes 0 or 1; only mx_quantize and the plain GEMM entry points accept 1, and with
    it the K % 128 rule of 6- and 4-bit operands becomes K % 32."""
    lib = mx.lib()
    shape = (ctypes.c_int64 * 2)(128, 96)
    buf = np.zeros(1 << 16, np.uint8)
    p = buf.ctypes.data + (-buf.ctypes.data) % 256
    pad = mx.binding.mx_opts_t(mx.MX_F32, mx.MX_SCALES_SWIZZLED, None, 0, 1)
    bad = mx.binding.mx_opts_t(mx.MX_F32, mx.MX_SCALES_SWIZZLED, None, 0, 2)
    assert lib.mx_quantize(p, p, p, shape, 2, 1, 4, 0, ctypes.byref(bad)) == mx.MX_ERR_FMT
    assert lib.mx_gemm(p, p, p, p, p, 128, 128, 96, 4, 4, ctypes.byref(bad)) == mx.MX_ERR_FMT
    assert lib.mx_quantize(p + 4, p, p, shape, 2, 1, 4, 0, ctypes.byref(pad)) == mx.MX_ERR_ALIGN  # accepted up to here
    assert lib.mx_gemm(p, p, p, p, p, 128, 128, 48, 4, 4, ctypes.byref(pad)) == mx.MX_ERR_SHAPE   # K % 32 stays
    assert lib.mx_gemm(p, p, p, p, p + 4, 128, 128, 96, 4, 4, ctypes.byref(pad)) == mx.MX_ERR_ALIGN  # K = 96 passes the shape rules
    assert lib.mx_gemm(p, p, p, p, p + 4, 128, 128, 96, 4, 4, None) == mx.MX_ERR_SHAPE
    assert lib.mx_dequantize(p, p, p, shape, 2, 1, 4, ctypes.byref(pad)) == mx.MX_ERR_UNSUPPORTED
    assert lib.mx_quantize_dual(p, p, p, p, p, 128, 128, 4, 0, ctypes.byref(pad)) == mx.MX_ERR_UNSUPPORTED
    assert lib.mx_gemm_batched(p, p, p, p, p, 0, 2, 128, 128, 96, 4, 4, ctypes.byref(pad)) == mx.MX_ERR_UNSUPPORTED
    assert lib.mx_gemm_dense(p, p, p, p, p, 0, 128, 128, 96, 4, 4, ctypes.byref(pad), p, 1 << 20) == mx.MX_ERR_UNSUPPORTED
    assert lib.mx_quantize_host_static(p, p, p, shape, 2, 1, 4, 0, ctypes.byref(pad)) == mx.MX_ERR_UNSUPPORTED


def test_extents_whose_products_wrap_are_rejected():
    """Shapes whose element count wraps a 64-bit integer (2^32 x 2^32 has numel 0 mod 2^64) or is
    simply absurd must come back as MX_ERR_SHAPE / size 0 from every entry point that derives a
    byte count from the shape -- above all from the entry point whose staging area is a fixed
    array, where a wrapped count would pass the size check."""
    lib = mx.lib()
    buf = np.zeros(4096, np.uint8)
    p = buf.ctypes.data + (-buf.ctypes.data) % 256
    o = mx.binding.mx_opts_t(mx.MX_F32, mx.MX_SCALES_SWIZZLED, None, 0)
    for dims in ((1 << 32, 1 << 32), (1 << 62, 4), (3, 1 << 62), (1 << 31, 1 << 31, 1 << 31), (1 << 45, 32)):
        shape = (ctypes.c_int64 * len(dims))(*dims)
        nd = len(dims)
        for axis in range(nd):
            assert mx.mx_elems_bytes(list(dims), axis, 0) == 0, dims
            assert mx.mx_scales_bytes(list(dims), axis, 1) == 0, dims
            assert lib.mx_quantize_host_workspace_bytes(shape, nd, axis, 0, ctypes.byref(o)) == 0
            assert lib.mx_quantize(p, p, p, shape, nd, axis, 0, 0, ctypes.byref(o)) == mx.MX_ERR_SHAPE, dims
            assert lib.mx_quantize_host_static(p, p, p, shape, nd, axis, 0, 0, ctypes.byref(o)) == mx.MX_ERR_SHAPE, dims
            assert lib.mx_quantize_host(p, p, p, shape, nd, axis, 0, 0, ctypes.byref(o), p, 1 << 20) == mx.MX_ERR_SHAPE
            assert lib.mx_dequantize_host(p, p, p, shape, nd, axis, 0, ctypes.byref(o), p, 1 << 20) == mx.MX_ERR_SHAPE
        assert lib.mx_dequantize(p, p, p, shape, nd, nd - 1, 0, ctypes.byref(o)) == mx.MX_ERR_SHAPE, dims
    # large but legitimate extents still get their sizes
    assert mx.mx_elems_bytes([1 << 20, 1 << 20], 1, 4) == 1 << 39
    # a request just over the fixed staging array is a workspace error, not a shape error
    shape = (ctypes.c_int64 * 2)(4096, 4096)
    assert lib.mx_quantize_host_static(p, p, p, shape, 2, 1, 0, 0, ctypes.byref(o)) == mx.MX_ERR_WORKSPACE


def test_gemm_variants_argument_validation_without_gpu():
    """The GEMM entry points added beside mx_gemm reject bad arguments before any CUDA call."""
    lib = mx.lib()
    buf = np.zeros(4096, np.uint8)
    p = buf.ctypes.data + (-buf.ctypes.data) % 256
    F32, BF16 = mx.MX_F32, mx.MX_BF16
    gb = lib.mx_gemm_bf16
    assert gb(p, p, p, p, None, 128, 128, 128, 0, 0, None) == mx.MX_ERR_NULL
    assert gb(p, p, p, p, p, 128, 132, 128, 0, 0, None) == mx.MX_ERR_SHAPE   # BF16 rows of C: N % 8
    assert gb(p, p, p, p, p, 128, 128, 128, 5, 0, None) == mx.MX_ERR_UNSUPPORTED
    bt = lib.mx_gemm_batched
    assert bt(p, p, p, p, p, 7, 2, 128, 128, 128, 0, 0, None) == mx.MX_ERR_FMT       # output dtype
    assert bt(p, p, p, p, p, F32, 2, 100, 128, 128, 0, 0, None) == mx.MX_ERR_SHAPE   # whole tiles only
    assert bt(p, p, p, p, p, F32, -1, 128, 128, 128, 0, 0, None) == mx.MX_ERR_SHAPE
    assert bt(p, p, p, p, p, F32, 1 << 30, 128, 128, 128, 0, 0, None) == mx.MX_ERR_SHAPE
    assert bt(p, p, p, p, p, BF16, 0, 128, 128, 128, 0, 0, None) == mx.MX_OK         # empty batch
    ge = lib.mx_gemm_ex
    P = mx.binding.mx_gemm_plan_t
    assert ge(p, p, p, p, p, 128, 128, 128, 0, 0, None, None) == ge(p, p, p, p, p, 128, 128, 128, 0, 0, None, ctypes.byref(P(0, 0, -1, -1, 0)))
    assert ge(p, p, p, p, p, 128, 128, 128, 0, 0, None, ctypes.byref(P(2, 0, -1, -1, 0))) == mx.MX_ERR_FMT
    assert ge(p, p, p, p, p, 128, 128, 128, 0, 0, None, ctypes.byref(P(0, 320, -1, -1, 0))) == mx.MX_ERR_SHAPE
    assert ge(p, p, p, p, p, 128, 128, 128, 0, 0, None, ctypes.byref(P(0, 0, 129, -1, 0))) == mx.MX_ERR_SHAPE
    assert ge(p, p, p, p, p, 128, 128, 128, 0, 0, None, ctypes.byref(P(0, 0, -1, -2, 0))) == mx.MX_ERR_SHAPE
    assert ge(p, p, p, p, p, 128, 128, 128, 0, 0, None, ctypes.byref(P(0, 0, -1, -1, -5))) == mx.MX_ERR_SHAPE
    assert ge(p, p, p, p, p, 128, 132, 128, 0, 0, None, ctypes.byref(P(1, 0, -1, -1, 0))) == mx.MX_ERR_SHAPE  # BF16 rows: N % 8
    gq = lib.mx_gemm_quantize
    assert gq(p, p, p, p, None, p, 128, 128, 128, 0, 0, 0, 0, None) == mx.MX_ERR_NULL
    assert gq(p, p, p, p, p, None, 128, 128, 128, 0, 0, 0, 0, None) == mx.MX_ERR_NULL
    assert gq(p, p, p, p, p, p, 128, 128, 128, 0, 0, 6, 0, None) == mx.MX_ERR_FMT
    assert gq(p, p, p, p, p, p, 128, 128, 128, 0, 0, 0, 2, None) == mx.MX_ERR_FMT
    assert gq(p, p, p, p, p, p, 100, 128, 128, 0, 0, 0, 0, None) == mx.MX_ERR_SHAPE   # whole tiles only
    assert gq(p, p, p, p, p, p + 4, 128, 128, 128, 0, 0, 0, 0, None) == mx.MX_ERR_ALIGN
    gd = lib.mx_gemm_dense
    assert lib.mx_gemm_dense_workspace_bytes(128, 256, 512) == 2 * (128 + 256) * 512
    assert lib.mx_gemm_dense_workspace_bytes(-1, 256, 512) == 0
    assert gd(p, p, p, p, p, F32, 128, 128, 128, 5, 5, None, None, 0) == mx.MX_ERR_NULL        # no workspace
    assert gd(p, p, p, p, p, F32, 128, 128, 128, 5, 5, None, p, 1024) == mx.MX_ERR_WORKSPACE
    assert gd(p, p, p, p, p, F32, 128, 128, 48, 5, 5, None, p, 1 << 20) == mx.MX_ERR_SHAPE
    assert gd(p, p, p, p, p, 3, 128, 128, 128, 5, 5, None, p, 1 << 20) == mx.MX_ERR_FMT
    assert gd(p, p, p, p, p, F32, 128, 128, 128, 6, 5, None, p, 1 << 20) == mx.MX_ERR_FMT
    assert gd(p, p, p, p, p, F32, 0, 128, 128, 5, 5, None, None, 0) == mx.MX_OK                # nothing to do


def test_header_is_plain_c(tmp_path):
    """include/mx.h compiles as C99 on its own (the boundary is a C ABI: no C++ in the signatures)
    and a C program can link against the library and call a host-only helper."""
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        import pytest
        pytest.skip("no C compiler")
    src = tmp_path / "t.c"
    src.write_text('#include "mx.h"\n'
                   'int main(void) { mx_conv_t c; mx_opts_t o; (void)c; (void)o;\n'
                   '  return mx_fmt_bits(MX_E2M3) == 6 && mx_scale_offset(33, 5, 128, 8, MX_SCALES_SWIZZLED) == 512 + 16 + 4 + 1 ? 0 : 1; }\n')
    exe = tmp_path / "t"
    libdir = os.path.dirname(mx.LIB_PATH)
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-I", os.path.join(ROOT, "include"),
                           str(src), "-o", str(exe), "-L", libdir, "-lmx_b200", "-Wl,-rpath," + libdir])
    assert subprocess.call([str(exe)]) == 0
