"""Convolution as a dot product of MX operands: mx_quantize (channels) -> mx_im2col -> mx_gemm
against the oracle (quantize -> dequantize -> the convolution sum in FP64).  The gather itself is
index work and is compared bit for bit with a table the oracle builds."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2310_10537_b200 as mx
from gpu_util import Guarded

pytestmark = pytest.mark.gpu
TOL = 1e-5

CASES = [
    # N, H, W, C, Cout, kh, kw, stride, pad, dilation, fmt_x, fmt_w, layout of x's scales
    (2, 14, 14, 64, 128, 3, 3, (1, 1), (1, 1), (1, 1), 0, 0, 1),
    (1, 17, 13, 32, 128, 3, 3, (2, 2), (1, 1), (1, 1), 1, 0, 0),      # odd extents, stride 2, linear scales in
    (3, 9, 11, 128, 256, 1, 1, (1, 1), (0, 0), (1, 1), 0, 4, 1),      # pointwise
    (1, 12, 12, 128, 128, 5, 3, (1, 2), (2, 0), (2, 1), 2, 3, 1),     # 6-bit codes (K % 128), dilation, asymmetric
    (2, 8, 8, 128, 128, 3, 3, (1, 1), (1, 1), (1, 1), 4, 4, 0),       # FP4 both (K = 1152)
    (1, 30, 30, 96, 384, 3, 3, (1, 1), (0, 0), (1, 1), 0, 0, 1),      # M = 784: ragged row tiles
    (2, 20, 20, 32, 128, 3, 3, (1, 1), (1, 1), (1, 1), 0, 1, 1),      # C = 32: a K chunk spans four taps, K tail (288)
    (4, 28, 28, 256, 256, 3, 3, (1, 1), (1, 1), (1, 1), 0, 0, 1),     # 25 row tiles x 2 column tiles, 18 K chunks
    (2, 16, 16, 64, 136, 2, 2, (2, 2), (0, 0), (1, 1), 1, 4, 0),      # FP4 filter, Cout not a multiple of 128
    (1, 12, 12, 128, 128, 5, 3, (1, 2), (2, 0), (2, 1), 0, 0, 1),     # C % 128 == 0: codes through the im2col map; asymmetric filter, stride, padding, dilation
    (2, 15, 17, 128, 256, 3, 3, (2, 2), (1, 1), (1, 1), 1, 0, 0),     # im2col map, stride 2, odd extents, last tile crosses the batch end
    (3, 7, 9, 384, 128, 2, 4, (1, 1), (0, 2), (1, 1), 0, 2, 1),       # im2col map, three channel chunks per tap, 6-bit filter
    (8, 56, 56, 128, 256, 3, 3, (1, 1), (1, 1), (1, 1), 0, 0, 1),     # large enough for the 256 x 256 CTA-pair tiles (two waves)
    (5, 40, 40, 128, 320, 3, 3, (1, 1), (1, 1), (1, 1), 1, 0, 0),     # pair tiles ragged in M (8000 rows) and in Cout, linear scales in
    (6, 33, 31, 256, 256, 3, 3, (2, 2), (1, 1), (1, 1), 0, 4, 1),     # pair tiles, stride 2, FP4 filter
]


def _expected_gather(codes_in, scales_in_linear, src, C, bits):
    """Rows of the im2col operand from the oracle's codes [pixels, C*bits/8] and scales [pixels, C/32]."""
    M, taps = src.shape
    bpp = C * bits // 8
    cb = C // 32
    e = np.zeros((M, taps, bpp), np.uint8)
    s = np.zeros((M, taps, cb), np.uint8)
    ok = src >= 0
    e[ok] = codes_in[src[ok]]
    s[ok] = scales_in_linear[src[ok]]
    return e.reshape(M, taps * bpp), s.reshape(M, taps * cb)


@pytest.mark.parametrize("case", CASES)
def test_conv_matches_oracle(case):
    N, H, W, C, Cout, kh, kw, st, pd, dl, fx, fw, layout = case
    g = torch.Generator(device="cuda").manual_seed(N * H + C + Cout)
    x = torch.randn((N, H, W, C), generator=g, device="cuda") * torch.exp(torch.randn((N, H, W, 1), generator=g, device="cuda"))
    w = torch.randn((Cout, kh, kw, C), generator=g, device="cuda") * 0.05
    conv = mx.mx_conv_geometry(N, H, W, C, kh, kw, st, pd, dl)
    Ho, Wo = mx.mx_conv_out_hw(conv)
    assert (Ho, Wo) == O.conv_out_hw(H, W, kh, kw, st, pd, dl)
    M, K = N * Ho * Wo, kh * kw * C

    # product path
    ex, sx = mx.mx_quantize(x, 3, fx, layout=layout)
    ea, sa = mx.mx_im2col(ex, sx, conv, fx, layout=layout)
    ew, sw = mx.mx_quantize(w.view(Cout, K), 1, fw)
    g_out = Guarded(M * Cout * 4)
    y = g_out.view.view(torch.float32).view(M, Cout)
    mx.mx_gemm(ea, sa, ew, sw, M, Cout, K, fx, fw, out=y, check_status=True)
    torch.cuda.synchronize()
    g_out.check()

    # oracle: quantize both operands, then (a) the gather, bit for bit
    xo = x.cpu().numpy().reshape(N * H * W, C)
    wo = w.cpu().numpy().reshape(Cout, K)
    oex, osx = O.quantize(xo, 1, fx, O.RNE, O.LINEAR)
    oew, osw = O.quantize(wo, 1, fw, O.RNE, O.SWIZZLED)
    bits = O.fmt_bits(fx)
    src = O.im2col_source_pixels(N, H, W, kh, kw, st, pd, dl)
    want_e, want_s = _expected_gather(oex.reshape(N * H * W, C * bits // 8), osx.reshape(N * H * W, C // 32), src, C, bits)
    assert np.array_equal(ea.cpu().numpy().reshape(M, K * bits // 8), want_e), "gathered codes"
    kb = K // 32
    got_s = sa.cpu().numpy()
    want_sw = np.zeros(O.scales_bytes(M, kb, O.SWIZZLED), np.uint8)
    rows, cols = np.meshgrid(np.arange(M), np.arange(kb), indexing="ij")
    offs = np.array([O.scale_offset(int(r), int(c), M, kb, O.SWIZZLED) for r, c in zip(rows.ravel()[:4 * kb], cols.ravel()[:4 * kb])])
    # offsets by the closed form for all entries (the helper above spot-checks the first rows)
    kchunks = (kb + 3) // 4
    off_all = ((rows >> 7) * kchunks + (cols >> 2)) * 512 + (rows & 31) * 16 + ((rows >> 5) & 3) * 4 + (cols & 3)
    assert np.array_equal(off_all.ravel()[:4 * kb], offs)
    want_sw[off_all.ravel()] = want_s.ravel()
    assert np.array_equal(got_s, want_sw), "gathered scales (padding must be 0)"

    # (b) the convolution of the dequantized operands in FP64
    xq = O.dequantize(oex, osx, N * H * W, C, fx, O.F64, O.LINEAR).reshape(N, H, W, C)
    wq = O.dequantize(oew, osw, Cout, K, fw, O.F64, O.SWIZZLED).reshape(Cout, kh, kw, C)
    y64, s64 = O.conv2d_nhwc(xq, wq, st, pd, dl)
    err = np.abs(y.cpu().numpy().astype(np.float64).reshape(N, Ho, Wo, Cout) - y64)
    assert (err <= TOL * s64).all(), f"{int((err > TOL * s64).sum())} outputs beyond 1e-5 * S"

    # (c) the same convolution with the operand gathered inside the GEMM (8-bit activations)
    if O.fmt_bits(fx) == 8:
        g2 = Guarded(M * Cout * 4)
        y2 = g2.view.view(torch.float32).view(M, Cout)
        mx.mx_conv2d(ex, sx, ew, sw, conv, Cout, fx, fw, layout=layout, out=y2, check_status=True)
        torch.cuda.synchronize()
        g2.check()
        err2 = np.abs(y2.cpu().numpy().astype(np.float64).reshape(N, Ho, Wo, Cout) - y64)
        assert (err2 <= TOL * s64).all(), f"implicit: {int((err2 > TOL * s64).sum())} outputs beyond 1e-5 * S"
        assert torch.equal(y2, y), "the gathered operand must give the materialized operand's result bit for bit"
        yb = mx.mx_conv2d(ex, sx, ew, sw, conv, Cout, fx, fw, layout=layout, out_dtype=torch.bfloat16, check_status=True)
        assert torch.equal(yb, y2.to(torch.bfloat16))
    else:
        with pytest.raises(mx.MxError) as ei:
            mx.mx_conv2d(ex, sx, ew, sw, conv, Cout, fx, fw, layout=layout)
        assert ei.value.status == mx.MX_ERR_UNSUPPORTED


def test_im2col_errors():
    z = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    with pytest.raises(mx.MxError) as e:
        mx.mx_im2col(z, z, mx.mx_conv_geometry(1, 8, 8, 48, 3, 3), 0)          # C % 32
    assert e.value.status == mx.MX_ERR_SHAPE
    with pytest.raises(mx.MxError) as e:
        mx.mx_im2col(z, z, mx.mx_conv_geometry(1, 8, 8, 32, 3, 3), 2)          # 6-bit: C % 64
    assert e.value.status == mx.MX_ERR_SHAPE
    with pytest.raises(mx.MxError) as e:
        mx.mx_im2col(z, z, mx.mx_conv_geometry(1, 2, 2, 32, 3, 3), 0)          # filter larger than the image
    assert e.value.status == mx.MX_ERR_SHAPE
    with pytest.raises(mx.MxError) as e:
        mx.mx_im2col(z, z, mx.mx_conv_geometry(1, 8, 8, 32, 3, 3, stride=(0, 1)), 0)
    assert e.value.status == mx.MX_ERR_SHAPE
