"""GPU parity: MX tensors stored zero-extended to a multiple of 128 along the block axis
(mx_opts_t::pad_k128), which lets 6- and 4-bit operands with K % 128 != 0 into the block-scaled
GEMM (Section 4.1: the dot product over K; zero codes add nothing to it).

(a) mx_quantize with the option == the oracle's quantize of the zero-extended tensor, byte for byte;
(b) mx_gemm on such operands against the oracle's FP64 dot product of the UNPADDED oracle operands."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2310_10537_b200 as mx
from gpu_util import Guarded, to_oracle_input

pytestmark = pytest.mark.gpu
TOL = 1e-5
BF16_REL = 2.0 ** -8


def _zero_extended(x: torch.Tensor, axis: int) -> torch.Tensor:
    L = x.shape[axis]
    Lp = (L + 127) // 128 * 128
    shape = list(x.shape)
    shape[axis] = Lp
    z = torch.zeros(shape, dtype=x.dtype)
    z.narrow(axis, 0, L).copy_(x.cpu())
    return z


@pytest.mark.parametrize("fmt", [mx.MX_E4M3, mx.MX_E5M2, mx.MX_E3M2, mx.MX_E2M3, mx.MX_E2M1, mx.MX_INT8])
@pytest.mark.parametrize("shape,axis,dtype,layout,rounding", [
    ((130, 96), 1, torch.float32, mx.MX_SCALES_SWIZZLED, mx.MX_RNE),
    ((130, 96), 1, torch.bfloat16, mx.MX_SCALES_LINEAR, mx.MX_RHAZ),
    ((5, 100), 1, torch.float32, mx.MX_SCALES_SWIZZLED, mx.MX_RHAZ),     # partial block and padding
    ((160, 200), 0, torch.bfloat16, mx.MX_SCALES_SWIZZLED, mx.MX_RNE),   # strided axis
    ((3, 416, 7), 1, torch.float32, mx.MX_SCALES_LINEAR, mx.MX_RNE),
    ((64, 256), 1, torch.float32, mx.MX_SCALES_SWIZZLED, mx.MX_RNE),     # nothing to pad: the fast path
])
def test_quantize_zero_extended(fmt, shape, axis, dtype, layout, rounding):
    g = torch.Generator(device="cuda").manual_seed(sum(shape) + fmt)
    x = (torch.randn(shape, generator=g, device="cuda") *
         torch.exp(2 * torch.randn(shape[:1] + (1,) * (len(shape) - 1), generator=g, device="cuda"))).to(dtype)
    stored = list(shape)
    stored[axis] = (stored[axis] + 127) // 128 * 128
    ge = Guarded(mx.mx_elems_bytes(stored, axis, fmt))
    gs = Guarded(mx.mx_scales_bytes(stored, axis, layout))
    mx.mx_quantize(x, axis, fmt, rounding, layout, out=(ge.view, gs.view), pad_k128=True)
    torch.cuda.synchronize()
    ge.check()
    gs.check()
    want_e, want_s = O.quantize(to_oracle_input(_zero_extended(x, axis)), axis, fmt, rounding, layout)
    assert np.array_equal(ge.view.cpu().numpy(), want_e)
    assert np.array_equal(gs.view.cpu().numpy(), want_s)


@pytest.mark.parametrize("M,N,K,fa,fb,dt", [
    (64, 256, 96, 4, 4, torch.float32),        # E2M1 x E2M1, K = 96
    (200, 520, 96, 4, 0, torch.float32),
    (130, 264, 160, 2, 3, torch.bfloat16),     # 6-bit operands, K = 160
    (16, 1024, 224, 4, 2, torch.float32),      # few rows of A
    (700, 2048, 1056, 3, 4, torch.float32),    # two-CTA tiles, K = 8 * 128 + 32
    (256, 256, 96, 0, 1, torch.float32),       # 8-bit operands take the option too
    (128, 128, 32, 4, 4, torch.float32),       # one block
])
def test_gemm_on_zero_extended_operands(M, N, K, fa, fb, dt):
    g = torch.Generator(device="cuda").manual_seed(M + N + K)
    A = torch.randn((M, K), generator=g, device="cuda") * torch.exp(torch.randn((M, 1), generator=g, device="cuda"))
    B = torch.randn((N, K), generator=g, device="cuda") * 0.05
    ea, sa = mx.mx_quantize(A, 1, fa, pad_k128=True)
    eb, sb = mx.mx_quantize(B, 1, fb, pad_k128=True)
    esz = 2 if dt == torch.bfloat16 else 4
    g_out = Guarded(M * N * esz)
    C = g_out.view.view(dt).view(M, N)
    if dt == torch.bfloat16:
        mx.mx_gemm_bf16(ea, sa, eb, sb, M, N, K, fa, fb, out=C, check_status=True, pad_k128=True)
    else:
        mx.mx_gemm(ea, sa, eb, sb, M, N, K, fa, fb, out=C, check_status=True, pad_k128=True)
    torch.cuda.synchronize()
    g_out.check()
    # the oracle never sees the padding: its own operands of the K-long tensors, its own dot product
    oa, osa = O.quantize(to_oracle_input(A), 1, fa)
    ob, osb = O.quantize(to_oracle_input(B), 1, fb)
    c64, s = O.gemm(oa, osa, ob, osb, M, N, K, fa, fb)
    fac, rel = ((1.0 + BF16_REL, BF16_REL) if dt == torch.bfloat16 else (1.0, 0.0))
    got = C.double().cpu().numpy()
    assert (np.abs(got - c64) <= fac * TOL * s + np.abs(c64) * rel).all()
    # and the product equals the one over the explicitly zero-extended tensors, bit for bit
    Kp = (K + 127) // 128 * 128
    Az = torch.zeros((M, Kp), device="cuda")
    Az[:, :K] = A
    Bz = torch.zeros((N, Kp), device="cuda")
    Bz[:, :K] = B
    eaz, saz = mx.mx_quantize(Az, 1, fa)
    ebz, sbz = mx.mx_quantize(Bz, 1, fb)
    assert torch.equal(eaz, ea) and torch.equal(saz, sa) and torch.equal(ebz, eb) and torch.equal(sbz, sb)
    Cz = mx.mx_gemm_ex(eaz, saz, ebz, sbz, M, N, Kp, fa, fb, out_dtype=dt, check_status=True)
    assert torch.equal(Cz, C)


def test_sub_byte_operands_without_the_option_keep_the_k128_rule():
    ea = torch.zeros(128 * 96 // 2, dtype=torch.uint8, device="cuda")
    sa = torch.zeros(512, dtype=torch.uint8, device="cuda")
    with pytest.raises(mx.MxError) as e:
        mx.mx_gemm(ea, sa, ea, sa, 128, 128, 96, mx.MX_E2M1, mx.MX_E2M1)
    assert e.value.status == mx.MX_ERR_SHAPE
