"""ctypes loader for the CPU oracle (``mx_oracle.c``).

TEST INFRASTRUCTURE.  Only ``tests/``, ``__graft_entry__.smoke()`` and the CPU
baseline legs of ``bench.py`` may import this package; the product package never
does.  Every function but the last two marshals numpy arrays into the C routines,
which restate Section 2 (values of an MX block), Section 3 / Algorithm 1
(conversion) and Section 4.1 (dot product) of arXiv 2310.10537; the convolution
helpers at the end are the textbook definition written out in numpy (FP64).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mx_oracle.c")
_LIB = os.path.join(_HERE, "libmx_oracle.so")

E4M3, E5M2, E3M2, E2M3, E2M1, INT8 = range(6)
FORMATS = {"e4m3": E4M3, "e5m2": E5M2, "e3m2": E3M2, "e2m3": E2M3, "e2m1": E2M1, "int8": INT8}
RNE, RHAZ = 0, 1
F32, BF16, F64 = 0, 1, 2
LINEAR, SWIZZLED = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, -O2, OpenMP over rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-std=c11", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i64, u8p, vp, dp = ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p
        ci = ctypes.c_int
        L.oracle_fmt_bits.argtypes = [ci]
        L.oracle_fmt_emax.argtypes = [ci]
        L.oracle_fmt_max_normal.argtypes = [ci]
        L.oracle_fmt_max_normal.restype = ctypes.c_double
        L.oracle_threads.restype = ci
        L.oracle_encode_element.argtypes = [ctypes.c_double, ci, ci]
        L.oracle_encode_element.restype = ctypes.c_uint8
        L.oracle_decode_element.argtypes = [ctypes.c_uint8, ci]
        L.oracle_decode_element.restype = ctypes.c_double
        L.oracle_scales_bytes.argtypes = [i64, i64, ci]
        L.oracle_scales_bytes.restype = ctypes.c_size_t
        L.oracle_scale_offset.argtypes = [i64, i64, i64, i64, ci]
        L.oracle_scale_offset.restype = ctypes.c_size_t
        L.oracle_elems_bytes.argtypes = [i64, i64, ci]
        L.oracle_elems_bytes.restype = ctypes.c_size_t
        L.oracle_pack_codes.argtypes = [u8p, i64, ci, u8p]
        L.oracle_pack_codes.restype = None
        L.oracle_unpack_codes.argtypes = [u8p, i64, ci, u8p]
        L.oracle_unpack_codes.restype = None
        L.oracle_quantize_block.argtypes = [vp, ci, ci, u8p, u8p]
        L.oracle_quantize.argtypes = [vp, ci, i64, i64, i64, ci, ci, ci, u8p, u8p]
        L.oracle_dequantize.argtypes = [u8p, u8p, i64, i64, ci, ci, ci, vp]
        L.oracle_gemm.argtypes = [u8p, u8p, u8p, u8p, i64, i64, i64, ci, ci, ci, dp, dp]
        L.oracle_gemm_samples.argtypes = [u8p, u8p, u8p, u8p, i64, i64, i64, ci, ci, ci,
                                          vp, vp, i64, dp, dp]
        _lib = L
    return _lib


def _ptr(a: np.ndarray) -> int:
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data


def threads() -> int:
    return lib().oracle_threads()


def fmt_bits(fmt: int) -> int:
    return lib().oracle_fmt_bits(fmt)


def fmt_emax(fmt: int) -> int:
    return lib().oracle_fmt_emax(fmt)


def fmt_max_normal(fmt: int) -> float:
    return lib().oracle_fmt_max_normal(fmt)


def encode_element(r: float, fmt: int, rounding: int = RNE) -> int:
    return int(lib().oracle_encode_element(float(r), fmt, rounding))


def decode_element(code: int, fmt: int) -> float:
    return float(lib().oracle_decode_element(int(code) & 0xFF, fmt))


def scales_bytes(rows: int, kblocks: int, layout: int) -> int:
    return int(lib().oracle_scales_bytes(rows, kblocks, layout))


def scale_offset(row: int, kb: int, rows: int, kblocks: int, layout: int) -> int:
    return int(lib().oracle_scale_offset(row, kb, rows, kblocks, layout))


def pack_codes(codes: np.ndarray, fmt: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    out = np.zeros(codes.size * fmt_bits(fmt) // 8, dtype=np.uint8)
    lib().oracle_pack_codes(_ptr(codes), codes.size, fmt, _ptr(out))
    return out


def unpack_codes(packed: np.ndarray, n: int, fmt: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    out = np.zeros(n, dtype=np.uint8)
    lib().oracle_unpack_codes(_ptr(packed), n, fmt, _ptr(out))
    return out


def quantize_block(v32, fmt: int, rounding: int = RNE):
    """Algorithm 1 on one block of 32 FP32 values -> (codes[32], scale byte)."""
    v = np.ascontiguousarray(v32, dtype=np.float32)
    assert v.size == 32
    codes = np.zeros(32, dtype=np.uint8)
    sb = np.zeros(1, dtype=np.uint8)
    rc = lib().oracle_quantize_block(_ptr(v), fmt, rounding, _ptr(codes), _ptr(sb))
    assert rc == 0
    return codes, int(sb[0])


def _as_input(x: np.ndarray):
    """float32 arrays go in as FP32; uint16 arrays are taken as BF16 bit patterns."""
    x = np.ascontiguousarray(x)
    if x.dtype == np.float32:
        return x, F32
    if x.dtype == np.uint16:
        return x, BF16
    raise TypeError("oracle input must be float32 or uint16 (bf16 bits)")


def quantize(x: np.ndarray, axis: int, fmt: int, rounding: int = RNE, layout: int = SWIZZLED):
    """Quantize along ``axis``; returns (packed elems uint8, scales uint8), K-major."""
    x, dt = _as_input(x)
    axis %= x.ndim
    outer = int(np.prod(x.shape[:axis], dtype=np.int64))
    L = x.shape[axis]
    inner = int(np.prod(x.shape[axis + 1:], dtype=np.int64))
    rows = outer * inner
    kblocks = (L + 31) // 32     # a partial last block is padded with zero codes
    elems = np.zeros(rows * kblocks * 32 * fmt_bits(fmt) // 8, dtype=np.uint8)
    scales = np.zeros(scales_bytes(rows, kblocks, layout), dtype=np.uint8)
    rc = lib().oracle_quantize(_ptr(x), dt, outer, L, inner, fmt, rounding, layout,
                               _ptr(elems), _ptr(scales))
    if rc != 0:
        raise ValueError(f"oracle_quantize failed: {rc}")
    return elems, scales


def dequantize(elems: np.ndarray, scales: np.ndarray, rows: int, L: int, fmt: int,
               out_dtype: int = F32, layout: int = SWIZZLED) -> np.ndarray:
    """Returns float32, uint16 (bf16 bits) or float64 array of shape [rows, L]."""
    np_dt = {F32: np.float32, BF16: np.uint16, F64: np.float64}[out_dtype]
    out = np.zeros((rows, L), dtype=np_dt)
    elems = np.ascontiguousarray(elems, dtype=np.uint8)
    scales = np.ascontiguousarray(scales, dtype=np.uint8)
    rc = lib().oracle_dequantize(_ptr(elems), _ptr(scales), rows, L, fmt, layout, out_dtype,
                                 _ptr(out))
    if rc != 0:
        raise ValueError(f"oracle_dequantize failed: {rc}")
    return out


def gemm(A, sA, B, sB, M: int, N: int, K: int, fmtA: int, fmtB: int, layout: int = SWIZZLED):
    """Full FP64 product and the sum of absolute products: (C64[M,N], S[M,N])."""
    C = np.zeros((M, N), dtype=np.float64)
    S = np.zeros((M, N), dtype=np.float64)
    rc = lib().oracle_gemm(_ptr(np.ascontiguousarray(A)), _ptr(np.ascontiguousarray(sA)),
                           _ptr(np.ascontiguousarray(B)), _ptr(np.ascontiguousarray(sB)),
                           M, N, K, fmtA, fmtB, layout, _ptr(C), _ptr(S))
    if rc != 0:
        raise ValueError(f"oracle_gemm failed: {rc}")
    return C, S


def gemm_samples(A, sA, B, sB, M: int, N: int, K: int, fmtA: int, fmtB: int, ms, ns,
                 layout: int = SWIZZLED):
    """FP64 dot products at the listed (m, n) positions: (c[count], s[count])."""
    ms = np.ascontiguousarray(ms, dtype=np.int64)
    ns = np.ascontiguousarray(ns, dtype=np.int64)
    c = np.zeros(ms.size, dtype=np.float64)
    s = np.zeros(ms.size, dtype=np.float64)
    rc = lib().oracle_gemm_samples(_ptr(np.ascontiguousarray(A)), _ptr(np.ascontiguousarray(sA)),
                                   _ptr(np.ascontiguousarray(B)), _ptr(np.ascontiguousarray(sB)),
                                   M, N, K, fmtA, fmtB, layout, _ptr(ms), _ptr(ns), ms.size,
                                   _ptr(c), _ptr(s))
    if rc != 0:
        raise ValueError(f"oracle_gemm_samples failed: {rc}")
    return c, s


def conv_out_hw(H: int, W: int, kh: int, kw: int, stride, pad, dilation):
    """Output extent of a 2-D convolution with zero padding on both sides."""
    Ho = (H + 2 * pad[0] - dilation[0] * (kh - 1) - 1) // stride[0] + 1
    Wo = (W + 2 * pad[1] - dilation[1] * (kw - 1) - 1) // stride[1] + 1
    return Ho, Wo


def conv2d_nhwc(x: np.ndarray, w: np.ndarray, stride=(1, 1), pad=(0, 0), dilation=(1, 1)):
    """Convolution as the dot product it is (Section 4.1 lists it among the dot-product operations):
    y[n, ho, wo, co] = sum_{i, j, c} x[n, ho*s_h - p_h + i*d_h, wo*s_w - p_w + j*d_w, c] * w[co, i, j, c],
    with x = 0 outside the image.  x[N, H, W, C] and w[Cout, kh, kw, C] are the VALUES of the
    operands (for MX operands: their dequantized values in FP64).  Returns (y, s) in FP64, s being the
    same sum over absolute values (the scale of the accumulation-error bound)."""
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    N, H, W, C = x.shape
    Cout, kh, kw, Cw = w.shape
    assert C == Cw
    Ho, Wo = conv_out_hw(H, W, kh, kw, stride, pad, dilation)
    xp = np.zeros((N, H + 2 * pad[0], W + 2 * pad[1], C), dtype=np.float64)
    xp[:, pad[0]:pad[0] + H, pad[1]:pad[1] + W, :] = x
    y = np.zeros((N, Ho, Wo, Cout), dtype=np.float64)
    s = np.zeros_like(y)
    for i in range(kh):
        for j in range(kw):
            h0, w0 = i * dilation[0], j * dilation[1]
            patch = xp[:, h0:h0 + (Ho - 1) * stride[0] + 1:stride[0],
                       w0:w0 + (Wo - 1) * stride[1] + 1:stride[1], :]          # [N, Ho, Wo, C]
            y += patch @ w[:, i, j, :].T
            s += np.abs(patch) @ np.abs(w[:, i, j, :]).T
    return y, s


def im2col_source_pixels(N: int, H: int, W: int, kh: int, kw: int, stride=(1, 1), pad=(0, 0),
                         dilation=(1, 1)) -> np.ndarray:
    """For every output pixel m = (n, ho, wo) and filter tap t = (i, j): the index n*H*W + hi*W + wi
    of the input pixel that the tap reads, or -1 where it falls into the padding.  Shape [M, kh*kw]."""
    Ho, Wo = conv_out_hw(H, W, kh, kw, stride, pad, dilation)
    src = np.full((N * Ho * Wo, kh * kw), -1, dtype=np.int64)
    for n in range(N):
        for ho in range(Ho):
            for wo in range(Wo):
                m = (n * Ho + ho) * Wo + wo
                for i in range(kh):
                    for j in range(kw):
                        hi = ho * stride[0] - pad[0] + i * dilation[0]
                        wi = wo * stride[1] - pad[1] + j * dilation[1]
                        if 0 <= hi < H and 0 <= wi < W:
                            src[m, i * kw + j] = (n * H + hi) * W + wi
    return src
