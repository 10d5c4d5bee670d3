"""ctypes binding of ``libmx_b200.so`` (the C ABI declared in ``include/mx.h``).

Argument marshalling only: every function takes torch tensors (or raw
pointers), passes ``data_ptr()`` and the current CUDA stream to the C entry point
of the same name and raises :class:`MxError` on a nonzero status.  PyTorch owns
the memory; all arithmetic runs in the library's CUDA kernels.  If the shared
library is missing the import of this module fails -- there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmx_b200.so")

# enums of include/mx.h
MX_E4M3, MX_E5M2, MX_E3M2, MX_E2M3, MX_E2M1, MX_INT8 = range(6)
FORMATS = {"e4m3": MX_E4M3, "e5m2": MX_E5M2, "e3m2": MX_E3M2, "e2m3": MX_E2M3,
           "e2m1": MX_E2M1, "int8": MX_INT8}
MX_RNE, MX_RHAZ = 0, 1
MX_F32, MX_BF16 = 0, 1
MX_SCALES_LINEAR, MX_SCALES_SWIZZLED = 0, 1
MX_OK = 0
MX_ERR_NULL, MX_ERR_SHAPE, MX_ERR_FMT, MX_ERR_ALIGN = -1, -2, -3, -4
MX_ERR_UNSUPPORTED, MX_ERR_CUDA, MX_ERR_TIMEOUT, MX_ERR_WORKSPACE = -5, -6, -7, -8

EXPORTS = [
    "mx_fmt_bits", "mx_elems_bytes", "mx_scales_bytes", "mx_scale_offset", "mx_strerror",
    "mx_last_cuda_error", "mx_quantize", "mx_quantize_dual", "mx_dequantize", "mx_gemm",
    "mx_gemm_bf16", "mx_gemm_ex", "mx_gemm_batched", "mx_gemm_quantize", "mx_gemm_dense_workspace_bytes",
    "mx_gemm_dense", "mx_conv_out_h", "mx_conv_out_w", "mx_im2col", "mx_conv2d",
    "mx_quantize_host_async", "mx_dequantize_host_async", "mx_host_synchronize",
    "mx_quantize_host_workspace_bytes", "mx_quantize_host", "mx_quantize_host_static",
    "mx_dequantize_host_workspace_bytes", "mx_dequantize_host",
    "mx_gemm_host_workspace_bytes", "mx_gemm_host",
]


class mx_opts_t(ctypes.Structure):
    _fields_ = [("dtype", ctypes.c_int32), ("scale_layout", ctypes.c_int32),
                ("stream", ctypes.c_void_p), ("check_status", ctypes.c_int32),
                ("pad_k128", ctypes.c_int32)]


class mx_gemm_plan_t(ctypes.Structure):
    _fields_ = [("c_dtype", ctypes.c_int32), ("tile_n", ctypes.c_int32),
                ("few_rows_limit", ctypes.c_int32), ("drop_fill", ctypes.c_int32),
                ("wait_cycles", ctypes.c_int64)]


class mx_conv_t(ctypes.Structure):
    _fields_ = [("N", ctypes.c_int64), ("H", ctypes.c_int64), ("W", ctypes.c_int64), ("C", ctypes.c_int64),
                ("kh", ctypes.c_int32), ("kw", ctypes.c_int32),
                ("stride_h", ctypes.c_int32), ("stride_w", ctypes.c_int32),
                ("pad_h", ctypes.c_int32), ("pad_w", ctypes.c_int32),
                ("dil_h", ctypes.c_int32), ("dil_w", ctypes.c_int32)]


class MxError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib.mx_strerror(status).decode()
        if status in (MX_ERR_CUDA, MX_ERR_TIMEOUT):
            msg += ": " + _lib.mx_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} ({status})")


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python paper_2310_10537_b200/build.py` "
            "(the library has no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i64p, u8p = ctypes.c_void_p, ctypes.POINTER(ctypes.c_int64), ctypes.c_void_p
    ci, i64, sz = ctypes.c_int, ctypes.c_int64, ctypes.c_size_t
    op = ctypes.POINTER(mx_opts_t)
    lib.mx_fmt_bits.argtypes = [ci]
    lib.mx_elems_bytes.argtypes = [i64p, ci, ci, ci]
    lib.mx_elems_bytes.restype = sz
    lib.mx_scales_bytes.argtypes = [i64p, ci, ci, ci]
    lib.mx_scales_bytes.restype = sz
    lib.mx_scale_offset.argtypes = [i64, i64, i64, i64, ci]
    lib.mx_scale_offset.restype = sz
    lib.mx_strerror.argtypes = [ci]
    lib.mx_strerror.restype = ctypes.c_char_p
    lib.mx_last_cuda_error.restype = ctypes.c_char_p
    lib.mx_quantize.argtypes = [vp, vp, u8p, i64p, ci, ci, ci, ci, op]
    lib.mx_quantize_dual.argtypes = [vp, vp, u8p, vp, u8p, i64, i64, ci, ci, op]
    lib.mx_dequantize.argtypes = [vp, u8p, vp, i64p, ci, ci, ci, op]
    lib.mx_gemm.argtypes = [vp, u8p, vp, u8p, vp, i64, i64, i64, ci, ci, op]
    lib.mx_gemm_bf16.argtypes = [vp, u8p, vp, u8p, vp, i64, i64, i64, ci, ci, op]
    lib.mx_gemm_ex.argtypes = [vp, u8p, vp, u8p, vp, i64, i64, i64, ci, ci, op, ctypes.POINTER(mx_gemm_plan_t)]
    lib.mx_gemm_quantize.argtypes = [vp, u8p, vp, u8p, vp, u8p, i64, i64, i64, ci, ci, ci, ci, op]
    lib.mx_gemm_dense_workspace_bytes.argtypes = [i64, i64, i64]
    lib.mx_gemm_dense_workspace_bytes.restype = sz
    lib.mx_gemm_dense.argtypes = [vp, u8p, vp, u8p, vp, ci, i64, i64, i64, ci, ci, op, vp, sz]
    cp = ctypes.POINTER(mx_conv_t)
    lib.mx_conv_out_h.argtypes = [cp]
    lib.mx_conv_out_h.restype = i64
    lib.mx_conv_out_w.argtypes = [cp]
    lib.mx_conv_out_w.restype = i64
    lib.mx_im2col.argtypes = [vp, u8p, vp, u8p, cp, ci, op]
    lib.mx_conv2d.argtypes = [vp, u8p, vp, u8p, vp, ci, cp, i64, ci, ci, op]
    lib.mx_gemm_batched.argtypes = [vp, u8p, vp, u8p, vp, ci, i64, i64, i64, i64, ci, ci, op]
    lib.mx_quantize_host_workspace_bytes.argtypes = [i64p, ci, ci, ci, op]
    lib.mx_quantize_host_workspace_bytes.restype = sz
    lib.mx_quantize_host.argtypes = [vp, vp, u8p, i64p, ci, ci, ci, ci, op, vp, sz]
    lib.mx_quantize_host_async.argtypes = [vp, vp, u8p, i64p, ci, ci, ci, ci, op, vp, sz]
    lib.mx_host_synchronize.argtypes = []
    lib.mx_quantize_host_static.argtypes = [vp, vp, u8p, i64p, ci, ci, ci, ci, op]
    lib.mx_dequantize_host_workspace_bytes.argtypes = [i64p, ci, ci, ci, op]
    lib.mx_dequantize_host_workspace_bytes.restype = sz
    lib.mx_dequantize_host.argtypes = [vp, u8p, vp, i64p, ci, ci, ci, op, vp, sz]
    lib.mx_dequantize_host_async.argtypes = [vp, u8p, vp, i64p, ci, ci, ci, op, vp, sz]
    lib.mx_gemm_host_workspace_bytes.argtypes = [i64, i64, i64, ci, ci]
    lib.mx_gemm_host_workspace_bytes.restype = sz
    lib.mx_gemm_host.argtypes = [vp, u8p, vp, u8p, vp, i64, i64, i64, ci, ci, op, vp, sz]
    return lib


_lib = _load()


def lib() -> ctypes.CDLL:
    """The loaded C library (for callers that pass raw pointers)."""
    return _lib


def _shape_arr(shape: Sequence[int]):
    return (ctypes.c_int64 * len(shape))(*[int(s) for s in shape])


def _dtype_code(dt: torch.dtype) -> int:
    if dt == torch.float32:
        return MX_F32
    if dt == torch.bfloat16:
        return MX_BF16
    raise TypeError(f"unsupported float dtype {dt}")


def _opts(dtype: int, layout: int, check: bool = False, stream: Optional[int] = None,
          pad_k128: bool = False) -> mx_opts_t:
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    return mx_opts_t(dtype, layout, ctypes.c_void_p(stream), 1 if check else 0, 1 if pad_k128 else 0)


def _check(status: int, where: str) -> None:
    if status != MX_OK:
        raise MxError(status, where)


def mx_fmt_bits(fmt: int) -> int:
    return _lib.mx_fmt_bits(fmt)


def mx_elems_bytes(shape: Sequence[int], axis: int, fmt: int) -> int:
    return int(_lib.mx_elems_bytes(_shape_arr(shape), len(shape), axis, fmt))


def mx_scales_bytes(shape: Sequence[int], axis: int, layout: int = MX_SCALES_SWIZZLED) -> int:
    return int(_lib.mx_scales_bytes(_shape_arr(shape), len(shape), axis, layout))


def mx_scale_offset(row: int, kblock: int, rows: int, kblocks: int,
                    layout: int = MX_SCALES_SWIZZLED) -> int:
    return int(_lib.mx_scale_offset(row, kblock, rows, kblocks, layout))


def mx_quantize(x: torch.Tensor, axis: int, fmt: int, rounding: int = MX_RNE,
                layout: int = MX_SCALES_SWIZZLED,
                out: Optional[Tuple[torch.Tensor, torch.Tensor]] = None,
                pad_k128: bool = False) -> Tuple[torch.Tensor, torch.Tensor]:
    """Quantize a contiguous CUDA tensor along ``axis`` (Algorithm 1).

    Returns (elems, scales) as flat uint8 tensors; the packed tensor has the
    quantization axis innermost.  ``out`` lets the caller reuse buffers.  ``pad_k128``: the
    result is the MX tensor of x zero-extended along ``axis`` to a multiple of 128."""
    assert x.is_cuda and x.is_contiguous()
    axis %= x.dim()
    shape = list(x.shape)
    if out is None:
        stored = list(shape)
        if pad_k128:
            stored[axis] = (stored[axis] + 127) // 128 * 128
        elems = torch.empty(mx_elems_bytes(stored, axis, fmt), dtype=torch.uint8, device=x.device)
        scales = torch.empty(mx_scales_bytes(stored, axis, layout), dtype=torch.uint8, device=x.device)
    else:
        elems, scales = out
    o = _opts(_dtype_code(x.dtype), layout, pad_k128=pad_k128)
    _check(_lib.mx_quantize(x.data_ptr(), elems.data_ptr(), scales.data_ptr(), _shape_arr(shape),
                            len(shape), axis, fmt, rounding, ctypes.byref(o)), "mx_quantize")
    return elems, scales


def mx_quantize_dual(x: torch.Tensor, fmt: int, rounding: int = MX_RNE, layout: int = MX_SCALES_SWIZZLED,
                     out=None, check_status: bool = False):
    """Both MX tensors of a contiguous 2-D CUDA tensor in one pass: returns
    ((elems_row, scales_row), (elems_col, scales_col)) = (mx_quantize(x, 1), mx_quantize(x, 0)).
    ``check_status``: synchronise and raise if a device-side wait of the kernel gave up."""
    assert x.is_cuda and x.is_contiguous() and x.dim() == 2
    R, C = x.shape
    if out is None:
        u8 = dict(dtype=torch.uint8, device=x.device)
        er = torch.empty(mx_elems_bytes([R, C], 1, fmt), **u8)
        sr = torch.empty(mx_scales_bytes([R, C], 1, layout), **u8)
        ec = torch.empty(mx_elems_bytes([R, C], 0, fmt), **u8)
        sc = torch.empty(mx_scales_bytes([R, C], 0, layout), **u8)
    else:
        (er, sr), (ec, sc) = out
    o = _opts(_dtype_code(x.dtype), layout, check=check_status)
    _check(_lib.mx_quantize_dual(x.data_ptr(), er.data_ptr(), sr.data_ptr(), ec.data_ptr(), sc.data_ptr(),
                                 R, C, fmt, rounding, ctypes.byref(o)), "mx_quantize_dual")
    return (er, sr), (ec, sc)


def mx_dequantize(elems: torch.Tensor, scales: torch.Tensor, shape: Sequence[int], fmt: int,
                  dtype: torch.dtype = torch.float32, layout: int = MX_SCALES_SWIZZLED,
                  out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Dequantize a packed MX tensor of logical shape ``shape`` (blocks along the last axis)."""
    assert elems.is_cuda and scales.is_cuda
    shape = list(shape)
    if out is None:
        out = torch.empty(shape, dtype=dtype, device=elems.device)
    o = _opts(_dtype_code(out.dtype), layout)
    _check(_lib.mx_dequantize(elems.data_ptr(), scales.data_ptr(), out.data_ptr(),
                              _shape_arr(shape), len(shape), len(shape) - 1, fmt,
                              ctypes.byref(o)), "mx_dequantize")
    return out


def mx_gemm(A: torch.Tensor, sA: torch.Tensor, B: torch.Tensor, sB: torch.Tensor,
            M: int, N: int, K: int, fmtA: int, fmtB: int,
            out: Optional[torch.Tensor] = None, check_status: bool = False,
            pad_k128: bool = False) -> torch.Tensor:
    """C[M,N] = A[M,K] . B[N,K]^T on MX operands (swizzled scales), FP32 output.  ``pad_k128``:
    both operands were written by mx_quantize with the same option (K % 32 == 0 then suffices)."""
    assert A.is_cuda and B.is_cuda and sA.is_cuda and sB.is_cuda
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32, device=A.device)
    o = _opts(MX_F32, MX_SCALES_SWIZZLED, check=check_status, pad_k128=pad_k128)
    _check(_lib.mx_gemm(A.data_ptr(), sA.data_ptr(), B.data_ptr(), sB.data_ptr(), out.data_ptr(),
                        M, N, K, fmtA, fmtB, ctypes.byref(o)), "mx_gemm")
    return out


def mx_gemm_bf16(A: torch.Tensor, sA: torch.Tensor, B: torch.Tensor, sB: torch.Tensor,
                 M: int, N: int, K: int, fmtA: int, fmtB: int,
                 out: Optional[torch.Tensor] = None, check_status: bool = False,
                 pad_k128: bool = False) -> torch.Tensor:
    """mx_gemm with the FP32 accumulator rounded to nearest even into a BF16 output."""
    assert A.is_cuda and B.is_cuda and sA.is_cuda and sB.is_cuda
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=A.device)
    assert out.dtype == torch.bfloat16
    o = _opts(MX_F32, MX_SCALES_SWIZZLED, check=check_status, pad_k128=pad_k128)
    _check(_lib.mx_gemm_bf16(A.data_ptr(), sA.data_ptr(), B.data_ptr(), sB.data_ptr(),
                             out.data_ptr(), M, N, K, fmtA, fmtB, ctypes.byref(o)), "mx_gemm_bf16")
    return out


def mx_gemm_ex(A: torch.Tensor, sA: torch.Tensor, B: torch.Tensor, sB: torch.Tensor,
               M: int, N: int, K: int, fmtA: int, fmtB: int, out: Optional[torch.Tensor] = None,
               out_dtype: torch.dtype = torch.float32, tile_n: int = 0, few_rows_limit: int = -1,
               wait_cycles: int = 0, drop_fill: int = -1, check_status: bool = False,
               pad_k128: bool = False) -> torch.Tensor:
    """mx_gemm / mx_gemm_bf16 with the kernel selection (tile_n, few_rows_limit) and the device-side
    wait budget (wait_cycles; drop_fill is the failure drill) in the caller's hands."""
    assert A.is_cuda and B.is_cuda and sA.is_cuda and sB.is_cuda
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=A.device)
    o = _opts(MX_F32, MX_SCALES_SWIZZLED, check=check_status, pad_k128=pad_k128)
    plan = mx_gemm_plan_t(_dtype_code(out.dtype), tile_n, few_rows_limit, drop_fill, wait_cycles)
    _check(_lib.mx_gemm_ex(A.data_ptr(), sA.data_ptr(), B.data_ptr(), sB.data_ptr(), out.data_ptr(),
                           M, N, K, fmtA, fmtB, ctypes.byref(o), ctypes.byref(plan)), "mx_gemm_ex")
    return out


def mx_gemm_batched(A: torch.Tensor, sA: torch.Tensor, B: torch.Tensor, sB: torch.Tensor,
                    batch: int, M: int, N: int, K: int, fmtA: int, fmtB: int,
                    out: Optional[torch.Tensor] = None, out_dtype: torch.dtype = torch.float32,
                    check_status: bool = False) -> torch.Tensor:
    """C[b] = A[b] . B[b]^T for b < batch; operands are the MX tensors of [batch, M, K] and
    [batch, N, K] quantized along K (swizzled scales)."""
    assert A.is_cuda and B.is_cuda and sA.is_cuda and sB.is_cuda
    if out is None:
        out = torch.empty((batch, M, N), dtype=out_dtype, device=A.device)
    o = _opts(MX_F32, MX_SCALES_SWIZZLED, check=check_status)
    _check(_lib.mx_gemm_batched(A.data_ptr(), sA.data_ptr(), B.data_ptr(), sB.data_ptr(),
                                out.data_ptr(), _dtype_code(out.dtype), batch, M, N, K, fmtA, fmtB,
                                ctypes.byref(o)), "mx_gemm_batched")
    return out


def mx_gemm_quantize(A: torch.Tensor, sA: torch.Tensor, B: torch.Tensor, sB: torch.Tensor,
                     M: int, N: int, K: int, fmtA: int, fmtB: int, fmtC: int, rounding: int = MX_RNE,
                     elems: Optional[torch.Tensor] = None, scales: Optional[torch.Tensor] = None,
                     check_status: bool = False) -> Tuple[torch.Tensor, torch.Tensor]:
    """A . B^T quantized along N in the GEMM epilogue: the MX tensor (codes, swizzled scales)
    mx_quantize would produce from the FP32 result."""
    assert A.is_cuda and B.is_cuda and sA.is_cuda and sB.is_cuda
    if elems is None:
        elems = torch.empty(M * N * mx_fmt_bits(fmtC) // 8, dtype=torch.uint8, device=A.device)
    if scales is None:
        scales = torch.empty(mx_scales_bytes((M, N), 1, MX_SCALES_SWIZZLED), dtype=torch.uint8,
                             device=A.device)
    o = _opts(MX_F32, MX_SCALES_SWIZZLED, check=check_status)
    _check(_lib.mx_gemm_quantize(A.data_ptr(), sA.data_ptr(), B.data_ptr(), sB.data_ptr(),
                                 elems.data_ptr(), scales.data_ptr(), M, N, K, fmtA, fmtB, fmtC,
                                 rounding, ctypes.byref(o)), "mx_gemm_quantize")
    return elems, scales


def mx_gemm_dense_workspace_bytes(M: int, N: int, K: int) -> int:
    return int(_lib.mx_gemm_dense_workspace_bytes(M, N, K))


def mx_gemm_dense(A: torch.Tensor, sA: torch.Tensor, B: torch.Tensor, sB: torch.Tensor,
                  M: int, N: int, K: int, fmtA: int, fmtB: int,
                  workspace: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None,
                  out_dtype: torch.dtype = torch.float32, check_status: bool = False) -> torch.Tensor:
    """A . B^T through BF16: dequantize both operands into ``workspace`` and run the dense BF16
    tensor-core GEMM (any format pair, MXINT8 included)."""
    assert A.is_cuda and B.is_cuda and sA.is_cuda and sB.is_cuda
    if workspace is None:
        workspace = torch.empty(mx_gemm_dense_workspace_bytes(M, N, K), dtype=torch.uint8, device=A.device)
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=A.device)
    o = _opts(MX_F32, MX_SCALES_SWIZZLED, check=check_status)
    _check(_lib.mx_gemm_dense(A.data_ptr(), sA.data_ptr(), B.data_ptr(), sB.data_ptr(), out.data_ptr(),
                              _dtype_code(out.dtype), M, N, K, fmtA, fmtB, ctypes.byref(o),
                              workspace.data_ptr(), workspace.numel()), "mx_gemm_dense")
    return out


def mx_conv_geometry(N: int, H: int, W: int, C: int, kh: int, kw: int, stride=(1, 1), pad=(0, 0),
                     dilation=(1, 1)) -> mx_conv_t:
    return mx_conv_t(N, H, W, C, kh, kw, stride[0], stride[1], pad[0], pad[1], dilation[0], dilation[1])


def mx_conv_out_hw(conv: mx_conv_t) -> Tuple[int, int]:
    return int(_lib.mx_conv_out_h(ctypes.byref(conv))), int(_lib.mx_conv_out_w(ctypes.byref(conv)))


def mx_im2col(elems: torch.Tensor, scales: torch.Tensor, conv: mx_conv_t, fmt: int,
              layout: int = MX_SCALES_SWIZZLED) -> Tuple[torch.Tensor, torch.Tensor]:
    """The MX tensor of x[N, H, W, C] (quantized along C) laid out as the K-major operand
    [N*Ho*Wo x kh*kw*C] of mx_gemm: (codes, swizzled scales)."""
    assert elems.is_cuda and scales.is_cuda
    Ho, Wo = mx_conv_out_hw(conv)
    M, K = conv.N * Ho * Wo, conv.kh * conv.kw * conv.C
    out_e = torch.empty(M * K * mx_fmt_bits(fmt) // 8, dtype=torch.uint8, device=elems.device)
    out_s = torch.empty(mx_scales_bytes((M, K), 1, MX_SCALES_SWIZZLED), dtype=torch.uint8, device=elems.device)
    o = _opts(MX_F32, layout)
    _check(_lib.mx_im2col(elems.data_ptr(), scales.data_ptr(), out_e.data_ptr(), out_s.data_ptr(),
                          ctypes.byref(conv), fmt, ctypes.byref(o)), "mx_im2col")
    return out_e, out_s


def mx_conv2d(x_elems: torch.Tensor, x_scales: torch.Tensor, w_elems: torch.Tensor, w_scales: torch.Tensor,
              conv: mx_conv_t, Cout: int, fmt_x: int, fmt_w: int, layout: int = MX_SCALES_SWIZZLED,
              out: Optional[torch.Tensor] = None, out_dtype: torch.dtype = torch.float32,
              check_status: bool = False) -> torch.Tensor:
    """y[N*Ho*Wo, Cout] = the convolution of the MX activation (quantized along C, 8-bit codes, scales
    in `layout`) with the MX filter [Cout x kh*kw*C], the im2col operand gathered inside the GEMM."""
    assert x_elems.is_cuda and x_scales.is_cuda and w_elems.is_cuda and w_scales.is_cuda
    Ho, Wo = mx_conv_out_hw(conv)
    M = conv.N * Ho * Wo
    if out is None:
        out = torch.empty((M, Cout), dtype=out_dtype, device=x_elems.device)
    o = _opts(MX_F32, layout, check=check_status)
    _check(_lib.mx_conv2d(x_elems.data_ptr(), x_scales.data_ptr(), w_elems.data_ptr(), w_scales.data_ptr(),
                          out.data_ptr(), _dtype_code(out.dtype), ctypes.byref(conv), Cout, fmt_x, fmt_w,
                          ctypes.byref(o)), "mx_conv2d")
    return out


# ---- host-buffer variants: tensors live in (pinned) host memory ----------------

def mx_quantize_host_workspace_bytes(shape, axis, fmt, dtype, layout=MX_SCALES_SWIZZLED) -> int:
    o = _opts(_dtype_code(dtype), layout, stream=0)
    return int(_lib.mx_quantize_host_workspace_bytes(_shape_arr(shape), len(shape), axis, fmt,
                                                     ctypes.byref(o)))


def mx_quantize_host(x: torch.Tensor, elems: torch.Tensor, scales: torch.Tensor, axis: int,
                     fmt: int, rounding: int, workspace: torch.Tensor,
                     layout: int = MX_SCALES_SWIZZLED, queue: bool = False) -> None:
    """Host tensors in and out.  ``queue=True`` uses the asynchronous entry point: the call only
    queues its work (own workspace per queued call) and ``mx_host_synchronize()`` waits for it."""
    assert not x.is_cuda and not elems.is_cuda and not scales.is_cuda and workspace.is_cuda
    shape = list(x.shape)
    o = _opts(_dtype_code(x.dtype), layout)
    fn = _lib.mx_quantize_host_async if queue else _lib.mx_quantize_host
    _check(fn(x.data_ptr(), elems.data_ptr(), scales.data_ptr(),
                                 _shape_arr(shape), len(shape), axis % len(shape), fmt, rounding,
                                 ctypes.byref(o), workspace.data_ptr(), workspace.numel()),
           "mx_quantize_host")


MX_STATIC_SCRATCH_BYTES = 16 * 1024 * 1024


def mx_quantize_host_static(x: torch.Tensor, elems: torch.Tensor, scales: torch.Tensor, axis: int,
                            fmt: int, rounding: int, layout: int = MX_SCALES_SWIZZLED) -> None:
    """mx_quantize_host for callers that may not allocate device memory: the staging area is a
    fixed array inside the library (MX_STATIC_SCRATCH_BYTES), so no workspace is passed.  Calls
    on one device share that array and must not overlap."""
    assert not x.is_cuda and not elems.is_cuda and not scales.is_cuda
    shape = list(x.shape)
    o = _opts(_dtype_code(x.dtype), layout)
    _check(_lib.mx_quantize_host_static(x.data_ptr(), elems.data_ptr(), scales.data_ptr(),
                                        _shape_arr(shape), len(shape), axis % len(shape), fmt,
                                        rounding, ctypes.byref(o)), "mx_quantize_host_static")


def mx_dequantize_host_workspace_bytes(shape, fmt, dtype, layout=MX_SCALES_SWIZZLED) -> int:
    o = _opts(_dtype_code(dtype), layout, stream=0)
    return int(_lib.mx_dequantize_host_workspace_bytes(_shape_arr(shape), len(shape),
                                                       len(shape) - 1, fmt, ctypes.byref(o)))


def mx_host_synchronize() -> None:
    """Waits for every queued host-buffer call on the current device."""
    _check(_lib.mx_host_synchronize(), "mx_host_synchronize")


def mx_dequantize_host(elems: torch.Tensor, scales: torch.Tensor, out: torch.Tensor, fmt: int,
                       workspace: torch.Tensor, layout: int = MX_SCALES_SWIZZLED, queue: bool = False) -> None:
    assert not elems.is_cuda and not scales.is_cuda and not out.is_cuda and workspace.is_cuda
    shape = list(out.shape)
    o = _opts(_dtype_code(out.dtype), layout)
    fn = _lib.mx_dequantize_host_async if queue else _lib.mx_dequantize_host
    _check(fn(elems.data_ptr(), scales.data_ptr(), out.data_ptr(),
                                   _shape_arr(shape), len(shape), len(shape) - 1, fmt,
                                   ctypes.byref(o), workspace.data_ptr(), workspace.numel()),
           "mx_dequantize_host")


def mx_gemm_host_workspace_bytes(M: int, N: int, K: int, fmtA: int, fmtB: int) -> int:
    return int(_lib.mx_gemm_host_workspace_bytes(M, N, K, fmtA, fmtB))


def mx_gemm_host(A, sA, B, sB, C, M: int, N: int, K: int, fmtA: int, fmtB: int,
                 workspace: torch.Tensor) -> None:
    assert not A.is_cuda and not C.is_cuda and workspace.is_cuda
    o = _opts(MX_F32, MX_SCALES_SWIZZLED)
    _check(_lib.mx_gemm_host(A.data_ptr(), sA.data_ptr(), B.data_ptr(), sB.data_ptr(),
                             C.data_ptr(), M, N, K, fmtA, fmtB, ctypes.byref(o),
                             workspace.data_ptr(), workspace.numel()), "mx_gemm_host")
