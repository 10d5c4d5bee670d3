"""GPU parity: mx_gemm through the C ABI against the CPU oracle.

Bound for every checked output (FP32 accumulation on the tensor cores against the
FP64 dot product of the same dequantized values):
    |C_gpu - C64| <= 1e-5 * sum_k |a_k| * |b_k|
Exactly representable cases must match exactly."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2310_10537_b200 as mx
import workloads as inputs
from gpu_util import Guarded, assert_operand_rows_match_oracle, to_oracle_input

pytestmark = pytest.mark.gpu
TOL = 1e-5
# BF16 output: the FP32 accumulator c32 obeys |c32 - c64| <= TOL * S and is rounded once to nearest
# even, |c_bf16 - c32| <= 2^-8 |c32| (half an ulp of an 8-bit significand), hence
#   |c_bf16 - c64| <= (1 + 2^-8) * TOL * S + 2^-8 * |c64|.
# FP32 output is held to TOL * S as stated, with no factor.
BF16_REL = 2.0 ** -8


def _bound_terms(dt):
    """(factor on TOL * S, relative term on |c64|) for an output of type dt."""
    return (1.0 + BF16_REL, BF16_REL) if dt == torch.bfloat16 else (1.0, 0.0)
FP = [mx.MX_E4M3, mx.MX_E5M2, mx.MX_E3M2, mx.MX_E2M3, mx.MX_E2M1]


def _gemm_guarded(ea, sa, eb, sb, M, N, K, fa, fb):
    g = Guarded(M * N * 4)
    out = g.view.view(torch.float32).view(M, N)
    mx.mx_gemm(ea, sa, eb, sb, M, N, K, fa, fb, out=out, check_status=True)
    torch.cuda.synchronize()
    g.check()
    return out


def _check_bound(C, C64, S, what):
    C = C.astype(np.float64)
    err = np.abs(C - C64)
    bound = TOL * S
    ok = (err <= bound) | (np.isnan(C) & np.isnan(C64))
    if not ok.all():
        i = np.flatnonzero(~ok.reshape(-1))[0]
        raise AssertionError(f"{what}: {int((~ok).sum())} of {ok.size} outputs beyond 1e-5*S; first "
                             f"flat index {i}: got {C.reshape(-1)[i]!r} want {C64.reshape(-1)[i]!r} "
                             f"S {S.reshape(-1)[i]!r}")
    return float(np.nanmax(err / np.maximum(S, 1e-300)))


def _packed_from_codes(codes: np.ndarray, fmt: int) -> torch.Tensor:
    return torch.from_numpy(O.pack_codes(codes.reshape(-1), fmt)).cuda()


def _swizzle_scales(sc: np.ndarray) -> np.ndarray:
    rows, kb = sc.shape
    out = np.zeros(O.scales_bytes(rows, kb, O.SWIZZLED), np.uint8)
    for r in range(rows):
        for k in range(kb):
            out[O.scale_offset(r, k, rows, kb, O.SWIZZLED)] = sc[r, k]
    return out


ONE = {mx.MX_E4M3: 0x38, mx.MX_E5M2: 0x3C, mx.MX_E3M2: 0x0C, mx.MX_E2M3: 0x08, mx.MX_E2M1: 0x2}


@pytest.mark.parametrize("fa,fb", [(0, 0), (1, 1), (2, 3), (3, 2), (4, 4), (0, 4), (4, 0), (2, 0)])
@pytest.mark.parametrize("N", [256, 384])
def test_scale_identification_exact(fa, fb, N):
    """Every element is 1.0 and every (row, K-block) has its own power-of-two scale, so each
    output is an exact sum that names the scale pairs the hardware applied: this pins the
    operand tile layout, the swizzled scale layout and the per-MMA scale selection."""
    M, K = 256, 1024
    kb = K // 32
    rng = np.random.default_rng(fa * 7 + fb + N)
    for f in (fa, fb):
        assert O.decode_element(ONE[f], f) == 1.0
    a_codes = np.full((M, K), ONE[fa], np.uint8)
    b_codes = np.full((N, K), ONE[fb], np.uint8)
    # exponents within +-3: every partial sum fits FP32's 24 bits, so the result is exact
    sa = (127 + rng.integers(-3, 4, (M, kb))).astype(np.uint8)
    sb = (127 + rng.integers(-3, 4, (N, kb))).astype(np.uint8)
    sa_sw, sb_sw = _swizzle_scales(sa), _swizzle_scales(sb)
    ea, eb = O.pack_codes(a_codes.reshape(-1), fa), O.pack_codes(b_codes.reshape(-1), fb)
    C = _gemm_guarded(torch.from_numpy(ea).cuda(), torch.from_numpy(sa_sw).cuda(),
                      torch.from_numpy(eb).cuda(), torch.from_numpy(sb_sw).cuda(), M, N, K, fa, fb)
    C64, _ = O.gemm(ea, sa_sw, eb, sb_sw, M, N, K, fa, fb)
    want = 32.0 * (2.0 ** (sa.astype(np.float64) - 127)) @ (2.0 ** (sb.astype(np.float64) - 127)).T
    assert (C64 == want).all()
    assert (C.cpu().numpy().astype(np.float64) == C64).all()


@pytest.mark.parametrize("fa,fb", [(0, 0), (1, 4), (2, 3), (4, 4), (3, 0)])
@pytest.mark.parametrize("M,N", [(16, 256), (40, 384), (96, 19200)])
def test_scale_identification_few_rows(fa, fb, M, N):
    """The same probe for M <= 96, where the kernel swaps the operands' places in the MMA (rows of
    B on the M side): every (row, K-block) scale of either operand must still meet its own codes.
    N = 19200 gives 150 tiles, so some CTAs walk a second tile (ring wrap, second accumulator)."""
    K = 256
    kb = K // 32
    rng = np.random.default_rng(fa * 7 + fb + N + M)
    a_codes = np.full((M, K), ONE[fa], np.uint8)
    b_codes = np.full((N, K), ONE[fb], np.uint8)
    sa = (127 + rng.integers(-3, 4, (M, kb))).astype(np.uint8)
    sb = (127 + rng.integers(-3, 4, (N, kb))).astype(np.uint8)
    sa_sw, sb_sw = _swizzle_scales(sa), _swizzle_scales(sb)
    ea, eb = O.pack_codes(a_codes.reshape(-1), fa), O.pack_codes(b_codes.reshape(-1), fb)
    C = _gemm_guarded(torch.from_numpy(ea).cuda(), torch.from_numpy(sa_sw).cuda(),
                      torch.from_numpy(eb).cuda(), torch.from_numpy(sb_sw).cuda(), M, N, K, fa, fb)
    want = 32.0 * (2.0 ** (sa.astype(np.float64) - 127)) @ (2.0 ** (sb.astype(np.float64) - 127)).T
    assert (C.cpu().numpy().astype(np.float64) == want).all()


@pytest.mark.parametrize("fa,fb", [(0, 0), (1, 0), (2, 3), (3, 3), (4, 4), (0, 4), (4, 1)])
@pytest.mark.parametrize("M,N,K,dt", [(1, 512, 128, torch.float32), (5, 1000, 384, torch.bfloat16),
                                      (33, 640, 1024, torch.float32), (96, 264, 640, torch.bfloat16)])
def test_few_rows_against_oracle(M, N, K, fa, fb, dt):
    """M <= 96 (the swapped-operand kernel), every format pair, both output types, tails in M and N."""
    g = torch.Generator(device="cuda").manual_seed(M + N + K + 10 * fa + fb)
    A = torch.randn((M, K), generator=g, device="cuda") * torch.exp(torch.randn((M, 1), generator=g, device="cuda"))
    B = torch.randn((N, K), generator=g, device="cuda") * 0.05
    ea, sa = mx.mx_quantize(A, 1, fa)
    eb, sb = mx.mx_quantize(B, 1, fb)
    esz = 2 if dt == torch.bfloat16 else 4
    g_out = Guarded(M * N * esz)
    C = g_out.view.view(dt).view(M, N)
    if dt == torch.bfloat16:
        mx.mx_gemm_bf16(ea, sa, eb, sb, M, N, K, fa, fb, out=C, check_status=True)
    else:
        mx.mx_gemm(ea, sa, eb, sb, M, N, K, fa, fb, out=C, check_status=True)
    torch.cuda.synchronize()
    g_out.check()
    hea, hsa, heb, hsb = (t.cpu().numpy().reshape(-1) for t in (ea, sa, eb, sb))
    c64, s = O.gemm(hea, hsa, heb, hsb, M, N, K, fa, fb)
    fac, rel = _bound_terms(dt)
    assert (np.abs(C.double().cpu().numpy() - c64) <= fac * TOL * s + np.abs(c64) * rel).all()


@pytest.mark.parametrize("M,N,K,fa,fb", [(64, 1024, 512, 0, 0), (17, 19200, 256, 4, 1), (96, 640, 1024, 2, 3)])
def test_few_rows_kernel_equals_tiled_kernel(M, N, K, fa, fb):
    """The same product through the swapped-operand kernel and (mx_gemm_ex with the threshold
    pinned to 0) through the 128-row tiles: bit-identical outputs."""
    g = torch.Generator(device="cuda").manual_seed(M * N + K)
    A = torch.randn((M, K), generator=g, device="cuda")
    B = torch.randn((N, K), generator=g, device="cuda")
    ea, sa = mx.mx_quantize(A, 1, fa)
    eb, sb = mx.mx_quantize(B, 1, fb)
    C1 = mx.mx_gemm(ea, sa, eb, sb, M, N, K, fa, fb, check_status=True)
    C2 = mx.mx_gemm_ex(ea, sa, eb, sb, M, N, K, fa, fb, few_rows_limit=0, check_status=True)
    torch.cuda.synchronize()
    assert torch.equal(C1, C2)
    assert C1.abs().max().item() > 0


@pytest.mark.parametrize("fa,fb,K", [(0, 0, 1024), (4, 4, 1024), (4, 4, 768), (2, 4, 512)])
def test_scale_identification_two_cta_kernels(fa, fb, K):
    """The same exact probe at a shape that selects the two-CTA kernels: E4M3 x E4M3 and FP6 x FP4 on
    kind::mxf8f6f4, FP4 x FP4 on kind::mxf4 (K % 256 == 0: two scales per row and MMA) and FP4 x FP4
    with K % 256 != 0 (falls back to kind::mxf8f6f4)."""
    M, N = 512, 256 * 37
    kb = K // 32
    rng = np.random.default_rng(fa * 7 + fb + K)
    a_codes = np.full((M, K), ONE[fa], np.uint8)
    b_codes = np.full((N, K), ONE[fb], np.uint8)
    sa = (127 + rng.integers(-3, 4, (M, kb))).astype(np.uint8)
    sb = (127 + rng.integers(-3, 4, (N, kb))).astype(np.uint8)
    sa_sw, sb_sw = _swizzle_scales(sa), _swizzle_scales(sb)
    ea, eb = O.pack_codes(a_codes.reshape(-1), fa), O.pack_codes(b_codes.reshape(-1), fb)
    C = _gemm_guarded(torch.from_numpy(ea).cuda(), torch.from_numpy(sa_sw).cuda(),
                      torch.from_numpy(eb).cuda(), torch.from_numpy(sb_sw).cuda(), M, N, K, fa, fb)
    want = 32.0 * (2.0 ** (sa.astype(np.float64) - 127)) @ (2.0 ** (sb.astype(np.float64) - 127)).T
    assert (C.cpu().numpy().astype(np.float64) == want).all()
    ms = rng.integers(0, M, 500)
    ns = rng.integers(0, N, 500)
    c64, _ = O.gemm_samples(ea, sa_sw, eb, sb_sw, M, N, K, fa, fb, ms, ns)
    assert (c64 == want[ms, ns]).all()


def test_element_position_probe_exact():
    """One nonzero element per row of A at a row-dependent K position against a B whose entries
    encode their K position: checks that element k of A meets element k of B for every k,
    across swizzle atoms, MMA K-slices and pipeline stages."""
    M = N = 128
    K = 512
    fa = fb = mx.MX_E4M3
    a_codes = np.zeros((M, K), np.uint8)
    for m in range(M):
        a_codes[m, (37 * m + 11) % K] = 0x38  # 1.0
    # B[n, k] = small integers that identify (n, k): value (k % 7 + 1) * sign(n)
    vals = np.array([[(k % 7 + 1) * (1 if (n + k) % 3 else -1) for k in range(K)] for n in range(N)], np.float32)
    b_codes = np.array([[O.encode_element(float(v), fb) for v in row] for row in vals], np.uint8)
    sa = np.full((M, K // 32), 127, np.uint8)
    sb = np.full((N, K // 32), 127, np.uint8)
    ea, eb = O.pack_codes(a_codes.reshape(-1), fa), O.pack_codes(b_codes.reshape(-1), fb)
    C = _gemm_guarded(torch.from_numpy(ea).cuda(), torch.from_numpy(_swizzle_scales(sa)).cuda(),
                      torch.from_numpy(eb).cuda(), torch.from_numpy(_swizzle_scales(sb)).cuda(),
                      M, N, K, fa, fb).cpu().numpy()
    want = np.array([[vals[n, (37 * m + 11) % K] for n in range(N)] for m in range(M)], np.float32)
    assert (C == want).all()


def test_config1_full_matrix():
    d = inputs.config1("cuda")
    A, B = d["A"], d["B"]
    M, K = A.shape
    N = B.shape[1]
    ea, sa = mx.mx_quantize(A, 1, mx.MX_E4M3)
    eb, sb = mx.mx_quantize(B, 0, mx.MX_E4M3)
    # operands are bit-exact against the oracle, so both sides multiply the same values
    wea, wsa = O.quantize(to_oracle_input(A), 1, O.E4M3)
    web, wsb = O.quantize(to_oracle_input(B), 0, O.E4M3)
    assert (ea.cpu().numpy() == wea).all() and (sa.cpu().numpy() == wsa).all()
    assert (eb.cpu().numpy() == web).all() and (sb.cpu().numpy() == wsb).all()
    C = _gemm_guarded(ea, sa, eb, sb, M, N, K, mx.MX_E4M3, mx.MX_E4M3)
    C64, S = O.gemm(wea, wsa, web, wsb, M, N, K, O.E4M3, O.E4M3)
    worst = _check_bound(C.cpu().numpy(), C64, S, "config 1")
    assert worst <= TOL
    # second launch gives the same bits (no order-dependent accumulation between launches)
    C2 = _gemm_guarded(ea, sa, eb, sb, M, N, K, mx.MX_E4M3, mx.MX_E4M3)
    assert torch.equal(C, C2)


@pytest.mark.parametrize("fa,fb", [(0, 0), (1, 0), (2, 3), (3, 3), (4, 4), (0, 4), (4, 1), (2, 2)])
@pytest.mark.parametrize("shape", [(128, 128, 128), (256, 384, 640), (384, 512, 1024)])
def test_all_format_pairs_small(fa, fb, shape):
    M, N, K = shape
    g = torch.Generator(device="cuda").manual_seed(M + N + K + fa * 11 + fb)
    A = torch.randn((M, K), generator=g, device="cuda") * torch.exp(torch.randn((M, 1), generator=g, device="cuda"))
    B = torch.randn((N, K), generator=g, device="cuda") * 0.05
    A.view(M, K // 32, 32)[::5, 1] = 0.0  # zero blocks contribute exactly nothing
    ea, sa = mx.mx_quantize(A, 1, fa, mx.MX_RHAZ)
    eb, sb = mx.mx_quantize(B, 1, fb, mx.MX_RNE)
    C = _gemm_guarded(ea, sa, eb, sb, M, N, K, fa, fb).cpu().numpy()
    C64, S = O.gemm(ea.cpu().numpy(), sa.cpu().numpy(), eb.cpu().numpy(), sb.cpu().numpy(), M, N, K, fa, fb)
    _check_bound(C, C64, S, (fa, fb, shape))


def test_long_k_accumulation_and_extreme_scales():
    M = N = 256
    K = 8192
    g = torch.Generator(device="cuda").manual_seed(99)
    A = torch.randn((M, K), generator=g, device="cuda")
    B = torch.randn((N, K), generator=g, device="cuda")
    # rows with very large and very small magnitudes: scale bytes far from 127
    A[:8] *= 2.0 ** 60
    A[8:16] *= 2.0 ** -60
    B[:8] *= 2.0 ** 40
    B[8:16] *= 2.0 ** -50
    for fa, fb in ((mx.MX_E4M3, mx.MX_E4M3), (mx.MX_E4M3, mx.MX_E2M1)):
        ea, sa = mx.mx_quantize(A, 1, fa)
        eb, sb = mx.mx_quantize(B, 1, fb)
        C = _gemm_guarded(ea, sa, eb, sb, M, N, K, fa, fb).cpu().numpy()
        C64, S = O.gemm(ea.cpu().numpy(), sa.cpu().numpy(), eb.cpu().numpy(), sb.cpu().numpy(), M, N, K, fa, fb)
        worst = _check_bound(C, C64, S, ("long K", fa, fb))
        print("long-K worst |err|/S:", worst)


def test_nan_scale_poisons_row_and_gemm_errors():
    M = N = 128
    K = 256
    g = torch.Generator(device="cuda").manual_seed(5)
    A = torch.randn((M, K), generator=g, device="cuda")
    B = torch.randn((N, K), generator=g, device="cuda")
    A[3, 40] = float("inf")   # block (3, 1) gets scale 0xFF
    B[7, 200] = float("nan")  # block (7, 6) gets scale 0xFF
    ea, sa = mx.mx_quantize(A, 1, mx.MX_E4M3)
    eb, sb = mx.mx_quantize(B, 1, mx.MX_E4M3)
    C = _gemm_guarded(ea, sa, eb, sb, M, N, K, 0, 0).cpu().numpy()
    C64, S = O.gemm(ea.cpu().numpy(), sa.cpu().numpy(), eb.cpu().numpy(), sb.cpu().numpy(), M, N, K, 0, 0)
    assert np.isnan(C64[3]).all() and np.isnan(C64[:, 7]).all()
    assert np.isnan(C[3]).all() and np.isnan(C[:, 7]).all()
    fin = ~np.isnan(C64)
    assert not np.isnan(C[fin]).any()
    _check_bound(np.where(fin, C, 0), np.where(fin, C64, 0), np.where(fin, S, 0), "finite part")
    with pytest.raises(mx.MxError) as ei:
        mx.mx_gemm(ea, sa, eb, sb, M, N, K - 16, 0, 0)
    assert ei.value.status == mx.MX_ERR_SHAPE
    with pytest.raises(mx.MxError) as ei:
        mx.mx_gemm(ea, sa, eb, sb, M, N, K, mx.MX_INT8, 0)
    assert ei.value.status == mx.MX_ERR_UNSUPPORTED


def _sample_positions(M, N, rng, full_rows=2, full_cols=2, tile=128):
    ms, ns = [], []
    for r in rng.choice(M, full_rows, replace=False):
        ms += [r] * N
        ns += list(range(N))
    for c in rng.choice(N, full_cols, replace=False):
        ms += list(range(M))
        ns += [c] * M
    tm, tn = M // tile, N // tile
    gm, gn = np.meshgrid(np.arange(tm), np.arange(tn), indexing="ij")
    ms += list((gm * tile + rng.integers(0, tile, gm.shape)).reshape(-1))
    ns += list((gn * tile + rng.integers(0, tile, gn.shape)).reshape(-1))
    ms += [0, 0, M - 1, M - 1]
    ns += [0, N - 1, 0, N - 1]
    return np.array(ms, np.int64), np.array(ns, np.int64)


def _full_size_check(name, ea, sa, eb, sb, M, N, K, fa, fb, seed):
    C = torch.empty((M, N), dtype=torch.float32, device="cuda")
    mx.mx_gemm(ea, sa, eb, sb, M, N, K, fa, fb, out=C, check_status=True)
    rng = np.random.default_rng(seed)
    ms, ns = _sample_positions(M, N, rng)
    hea, hsa, heb, hsb = (t.cpu().numpy() for t in (ea, sa, eb, sb))
    c64, s = O.gemm_samples(hea, hsa, heb, hsb, M, N, K, fa, fb, ms, ns)
    got = C[torch.from_numpy(ms).cuda(), torch.from_numpy(ns).cuda()].cpu().numpy()
    worst = _check_bound(got, c64, s, name + " sampled")
    # whole matrix against an FP64 library product of the oracle-dequantized operands
    da = torch.from_numpy(O.dequantize(hea, hsa, M, K, fa, O.F64)).cuda()
    db = torch.from_numpy(O.dequantize(heb, hsb, N, K, fb, O.F64)).cuda()
    rows_per = max(128, (1 << 27) // N // 128 * 128)
    bad = 0
    for r0 in range(0, M, rows_per):
        r1 = min(M, r0 + rows_per)
        c64f = da[r0:r1] @ db.T
        sf = da[r0:r1].abs() @ db.abs().T
        bad += int(((C[r0:r1].double() - c64f).abs() > TOL * sf).sum())
    assert bad == 0, f"{name}: {bad} outputs of the full matrix beyond the bound"
    print(name, "worst sampled |err|/S:", worst)


@pytest.mark.parametrize("shape,fa,fb", [
    ((4736, 8192, 256), 0, 0),    # M = 37 x 128: the one-CTA 128 x 256 kernel
    ((4736, 8320, 384), 3, 4),    # ... with a ragged last tile (N = 65 x 128)
    ((2048, 9600, 384), 0, 2),    # M % 256 == 0: the two-CTA 256 x 256 kernel, ragged N
    ((256, 256 * 74, 128), 1, 0),  # two-CTA kernel, one tile per pair, a single K stage
    ((2048, 9600, 512), 4, 4),    # FP4 x FP4 on kind::mxf4 (K % 256 == 0), ragged N
    ((256, 256 * 74, 256), 4, 4),  # kind::mxf4, a single K stage
    ((1024, 4864, 640), 4, 4),    # FP4 x FP4 with K % 256 != 0: kind::mxf8f6f4
])
def test_kernel_variants_whole_matrix(shape, fa, fb):
    """Shapes that select each GEMM kernel variant; the whole output is checked against an
    FP64 library product of the oracle-dequantized operands and sampled against the oracle."""
    M, N, K = shape
    g = torch.Generator(device="cuda").manual_seed(M + N + K)
    A = torch.randn((M, K), generator=g, device="cuda") * torch.exp(torch.randn((M, 1), generator=g, device="cuda"))
    B = torch.randn((N, K), generator=g, device="cuda") * 0.02
    ea, sa = mx.mx_quantize(A, 1, fa)
    eb, sb = mx.mx_quantize(B, 1, fb)
    g_out = Guarded(M * N * 4)
    C = g_out.view.view(torch.float32).view(M, N)
    mx.mx_gemm(ea, sa, eb, sb, M, N, K, fa, fb, out=C, check_status=True)
    torch.cuda.synchronize()
    g_out.check()
    hea, hsa, heb, hsb = (t.cpu().numpy() for t in (ea, sa, eb, sb))
    da = torch.from_numpy(O.dequantize(hea, hsa, M, K, fa, O.F64)).cuda()
    db = torch.from_numpy(O.dequantize(heb, hsb, N, K, fb, O.F64)).cuda()
    bad = int(((C.double() - da @ db.T).abs() > TOL * (da.abs() @ db.abs().T)).sum())
    assert bad == 0, f"{shape}: {bad} outputs beyond the bound"
    rng = np.random.default_rng(M)
    ms, ns = rng.integers(0, M, 2000), rng.integers(0, N, 2000)
    c64, s = O.gemm_samples(hea, hsa, heb, hsb, M, N, K, fa, fb, ms, ns)
    _check_bound(C[torch.from_numpy(ms).cuda(), torch.from_numpy(ns).cuda()].cpu().numpy(), c64, s, shape)


@pytest.mark.parametrize("shape,fa,fb", [
    ((384, 512, 1024), 0, 1),     # one-CTA 128 x 128 tiles
    ((4736, 8320, 384), 3, 4),    # one-CTA 128 x 256 tiles, ragged last tile
    ((2048, 9600, 384), 0, 2),    # two-CTA tiles, ragged N
    ((2048, 9600, 512), 4, 4),    # kind::mxf4
])
def test_bf16_output(shape, fa, fb):
    """mx_gemm_bf16 against the oracle: |C - exact| <= 1e-5 * S + 2^-8 |FP32 value| (half a
    BF16 ulp: one rounding of the FP32 accumulator, itself within 1e-5 * S of exact), on the whole matrix through an FP64 library
    product of the oracle-dequantized operands and on samples through the oracle's GEMM; the
    canary bytes around the output stay intact (a BF16 row is half as long as an FP32 one)."""
    M, N, K = shape
    g = torch.Generator(device="cuda").manual_seed(M * 3 + N + K)
    A = torch.randn((M, K), generator=g, device="cuda") * torch.exp(torch.randn((M, 1), generator=g, device="cuda"))
    B = torch.randn((N, K), generator=g, device="cuda") * 0.02
    ea, sa = mx.mx_quantize(A, 1, fa)
    eb, sb = mx.mx_quantize(B, 1, fb)
    g_out = Guarded(M * N * 2)
    C = g_out.view.view(torch.bfloat16).view(M, N)
    mx.mx_gemm_bf16(ea, sa, eb, sb, M, N, K, fa, fb, out=C, check_status=True)
    torch.cuda.synchronize()
    g_out.check()
    hea, hsa, heb, hsb = (t.cpu().numpy() for t in (ea, sa, eb, sb))
    da = torch.from_numpy(O.dequantize(hea, hsa, M, K, fa, O.F64)).cuda()
    db = torch.from_numpy(O.dequantize(heb, hsb, N, K, fb, O.F64)).cuda()
    ref = da @ db.T
    bound = (1.0 + BF16_REL) * TOL * (da.abs() @ db.abs().T) + ref.abs() * BF16_REL
    bad = int(((C.double() - ref).abs() > bound).sum())
    assert bad == 0, f"{shape}: {bad} outputs beyond the bound"
    rng = np.random.default_rng(N)
    ms, ns = rng.integers(0, M, 1000), rng.integers(0, N, 1000)
    c64, s = O.gemm_samples(hea, hsa, heb, hsb, M, N, K, fa, fb, ms, ns)
    got = C[torch.from_numpy(ms).cuda(), torch.from_numpy(ns).cuda()].double().cpu().numpy()
    assert (np.abs(got - c64) <= (1.0 + BF16_REL) * TOL * s + np.abs(c64) * BF16_REL).all()
    # the BF16 result is the FP32 result of the same kernel rounded once to nearest even
    C32 = mx.mx_gemm(ea, sa, eb, sb, M, N, K, fa, fb, check_status=True)
    assert torch.equal(C32.to(torch.bfloat16).view(torch.int16), C.view(torch.int16))


@pytest.mark.parametrize("batch,M,N,K,fa,fb,dt", [
    (24, 512, 512, 128, 0, 0, torch.float32),    # attention scores S x S over d = 128: two-CTA tiles
    (5, 384, 640, 256, 1, 3, torch.float32),     # one-CTA 128 x 128 tiles
    (40, 384, 640, 256, 0, 4, torch.float32),    # one-CTA 128 x 256 tiles, ragged tile reaching into the next matrix
    (30, 256, 384, 256, 4, 4, torch.bfloat16),   # kind::mxf4 pairs, ragged N, BF16 out
    (1, 256, 256, 128, 2, 2, torch.float32),
])
def test_batched(batch, M, N, K, fa, fb, dt):
    """mx_gemm_batched: every matrix of the batch against the oracle (the first and the last in
    full through the oracle's GEMM, all of them through an FP64 library product of the
    oracle-dequantized operands)."""
    g = torch.Generator(device="cuda").manual_seed(batch + M + N + K)
    A = torch.randn((batch, M, K), generator=g, device="cuda") * torch.exp(torch.randn((batch, M, 1), generator=g, device="cuda"))
    B = torch.randn((batch, N, K), generator=g, device="cuda") * torch.exp(torch.randn((batch, 1, 1), generator=g, device="cuda"))
    ea, sa = mx.mx_quantize(A, 2, fa)
    eb, sb = mx.mx_quantize(B, 2, fb)
    esz = 2 if dt == torch.bfloat16 else 4
    g_out = Guarded(batch * M * N * esz)
    C = g_out.view.view(dt).view(batch, M, N)
    mx.mx_gemm_batched(ea, sa, eb, sb, batch, M, N, K, fa, fb, out=C, check_status=True)
    torch.cuda.synchronize()
    g_out.check()
    hea, hsa, heb, hsb = (t.cpu().numpy().reshape(-1) for t in (ea, sa, eb, sb))
    da = torch.from_numpy(O.dequantize(hea, hsa, batch * M, K, fa, O.F64)).cuda().view(batch, M, K)
    db = torch.from_numpy(O.dequantize(heb, hsb, batch * N, K, fb, O.F64)).cuda().view(batch, N, K)
    ref = da @ db.transpose(1, 2)
    S = da.abs() @ db.abs().transpose(1, 2)
    fac, rel = _bound_terms(dt)
    bad = int(((C.double() - ref).abs() > fac * TOL * S + ref.abs() * rel).sum())
    assert bad == 0, f"{bad} outputs beyond the bound"
    abytes, bbytes = M * K * O.fmt_bits(fa) // 8, N * K * O.fmt_bits(fb) // 8
    for b in {0, batch - 1}:
        c64, s = O.gemm(hea[b * abytes:(b + 1) * abytes], hsa[b * M * K // 32:(b + 1) * M * K // 32],
                        heb[b * bbytes:(b + 1) * bbytes], hsb[b * N * K // 32:(b + 1) * N * K // 32],
                        M, N, K, fa, fb)
        got = C[b].double().cpu().numpy()
        assert (np.abs(got - c64) <= fac * TOL * s + np.abs(c64) * rel).all(), f"matrix {b}"


def test_batched_errors():
    z = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    out = torch.full((4,), 7.0, device="cuda")
    with pytest.raises(mx.MxError) as e:
        mx.mx_gemm_batched(z, z, z, z, -1, 128, 128, 128, 0, 0, out=out)
    assert e.value.status == mx.MX_ERR_SHAPE
    with pytest.raises(mx.MxError) as e:
        mx.mx_gemm_batched(z, z, z, z, 1 << 24, 128, 128, 128, 0, 0, out=out)
    assert e.value.status == mx.MX_ERR_SHAPE
    mx.mx_gemm_batched(z, z, z, z, 0, 128, 128, 128, 0, 0, out=out)   # batch 0: nothing written
    assert (out == 7.0).all()


@pytest.mark.parametrize("shape,fa,fb", [
    ((256, 512, 512), 0, 0),       # below the two-CTA threshold: one-CTA 128 x 128 tiles, two blocks per thread
    ((4736, 1024, 128), 1, 3),     # one-CTA 128 x 256 tiles
    ((2048, 2560, 256), 0, 2),     # two-CTA 256 x 256 tiles
    ((2048, 2560, 256), 4, 4),     # kind::mxf4
])
@pytest.mark.parametrize("fc,rounding", [(0, 0), (1, 1), (2, 0), (3, 1), (4, 0), (4, 1), (5, 0), (5, 1)])
def test_gemm_quantize_exact_operands(shape, fa, fb, fc, rounding):
    """mx_gemm_quantize against the oracle chain quantize -> gemm -> quantize, bit for bit, on
    operands whose dot products are exact in FP32 (so both sides quantize the same numbers; the
    results are integers of up to 15 bits, full of rounding ties for every element format)."""
    M, N, K = shape
    rng = np.random.default_rng(M + N + K + fa)
    rowexp = np.exp2(rng.integers(-1, 2, (M, 1))).astype(np.float32)
    A = rng.integers(-3, 4, (M, K)).astype(np.float32)
    B = rng.integers(-3, 4, (N, K)).astype(np.float32)
    A[:, ::32] = 3.0   # every block holds a 3: one shared exponent per row, every value kept exactly
    B[:, ::32] = -3.0
    A *= rowexp
    oa, osa = O.quantize(A, 1, fa)
    ob, osb = O.quantize(B, 1, fb)
    assert np.array_equal(O.dequantize(oa, osa, M, K, fa, O.F64), A.astype(np.float64))
    assert np.array_equal(O.dequantize(ob, osb, N, K, fb, O.F64), B.astype(np.float64))
    c64, _ = O.gemm(oa, osa, ob, osb, M, N, K, fa, fb)
    c32 = c64.astype(np.float32)
    assert np.array_equal(c32.astype(np.float64), c64)
    want_e, want_s = O.quantize(c32, 1, fc, rounding)

    ea, sa = mx.mx_quantize(torch.from_numpy(A).cuda(), 1, fa)
    eb, sb = mx.mx_quantize(torch.from_numpy(B).cuda(), 1, fb)
    assert np.array_equal(ea.cpu().numpy().reshape(-1), oa) and np.array_equal(sa.cpu().numpy().reshape(-1), osa)
    assert np.array_equal(eb.cpu().numpy().reshape(-1), ob) and np.array_equal(sb.cpu().numpy().reshape(-1), osb)
    ge = Guarded(want_e.size)
    gs = Guarded(want_s.size)
    mx.mx_gemm_quantize(ea, sa, eb, sb, M, N, K, fa, fb, fc, rounding, elems=ge.view, scales=gs.view,
                        check_status=True)
    torch.cuda.synchronize()
    ge.check()
    gs.check()
    assert np.array_equal(gs.view.cpu().numpy(), want_s), "scale bytes"
    got = ge.view.cpu().numpy()
    if not np.array_equal(got, want_e):
        i = int(np.flatnonzero(got != want_e)[0])
        raise AssertionError(f"{int((got != want_e).sum())} code bytes differ, first at byte {i}: "
                             f"got {got[i]:#x} want {want_e[i]:#x}")


@pytest.mark.parametrize("fc,rounding", [(0, 0), (2, 1), (4, 0), (5, 1)])
def test_gemm_quantize_equals_gemm_then_quantize(fc, rounding):
    """On general operands the fused call writes, bit for bit, what mx_quantize makes of mx_gemm's
    FP32 result (each of those two is checked against the oracle on its own); special values
    included: a NaN scale in A poisons a row of C, whose blocks must come out as scale 0xFF."""
    M, N, K = 2048, 2304, 512
    g = torch.Generator(device="cuda").manual_seed(7 + fc)
    A = torch.randn((M, K), generator=g, device="cuda") * torch.exp(2 * torch.randn((M, 1), generator=g, device="cuda"))
    B = torch.randn((N, K), generator=g, device="cuda") * torch.exp(torch.randn((N, 1), generator=g, device="cuda"))
    A[5, 40] = float("nan")
    A[300:302] = 0.0            # zero rows of C: zero blocks
    ea, sa = mx.mx_quantize(A, 1, 0)
    eb, sb = mx.mx_quantize(B, 1, 1)
    C = mx.mx_gemm(ea, sa, eb, sb, M, N, K, 0, 1, check_status=True)
    assert bool(torch.isnan(C[5]).all())
    we, ws = mx.mx_quantize(C, 1, fc, rounding)
    fe, fs = mx.mx_gemm_quantize(ea, sa, eb, sb, M, N, K, 0, 1, fc, rounding, check_status=True)
    assert torch.equal(fs.view(-1), ws.view(-1))
    assert torch.equal(fe.view(-1), we.view(-1))
    # and the oracle's quantization of that same FP32 matrix
    oe, osc = O.quantize(C.cpu().numpy(), 1, fc, rounding)
    assert np.array_equal(fe.cpu().numpy().reshape(-1), oe) and np.array_equal(fs.cpu().numpy().reshape(-1), osc)


@pytest.mark.parametrize("shape,fa,fb,dt", [
    ((384, 512, 1024), 5, 5, torch.float32),     # MXINT8 x MXINT8, one-CTA 128 x 128 tiles
    ((128, 128, 128), 5, 0, torch.float32),
    ((4736, 8320, 256), 5, 0, torch.float32),    # one-CTA 128 x 256 tiles, ragged last tile
    ((2048, 9600, 384), 0, 5, torch.float32),    # two-CTA tiles, ragged N
    ((2048, 9600, 384), 5, 5, torch.bfloat16),
    ((512, 640, 256), 2, 4, torch.float32),      # the BF16 route also takes the formats mx_gemm takes
])
def test_gemm_dense(shape, fa, fb, dt):
    """mx_gemm_dense (dequantize to BF16 + dense BF16 tensor-core GEMM; the MXINT8 route): whole
    matrix against an FP64 library product of the oracle-dequantized operands, samples against the
    oracle's GEMM, same bound as mx_gemm."""
    M, N, K = shape
    g = torch.Generator(device="cuda").manual_seed(M + 2 * N + K + fa)
    A = torch.randn((M, K), generator=g, device="cuda") * torch.exp(torch.randn((M, 1), generator=g, device="cuda"))
    B = torch.randn((N, K), generator=g, device="cuda") * 0.02
    ea, sa = mx.mx_quantize(A, 1, fa)
    eb, sb = mx.mx_quantize(B, 1, fb)
    esz = 2 if dt == torch.bfloat16 else 4
    g_out = Guarded(M * N * esz)
    g_ws = Guarded(mx.mx_gemm_dense_workspace_bytes(M, N, K))
    C = g_out.view.view(dt).view(M, N)
    mx.mx_gemm_dense(ea, sa, eb, sb, M, N, K, fa, fb, workspace=g_ws.view, out=C, check_status=True)
    torch.cuda.synchronize()
    g_out.check()
    g_ws.check()
    hea, hsa, heb, hsb = (t.cpu().numpy().reshape(-1) for t in (ea, sa, eb, sb))
    da = torch.from_numpy(O.dequantize(hea, hsa, M, K, fa, O.F64)).cuda()
    db = torch.from_numpy(O.dequantize(heb, hsb, N, K, fb, O.F64)).cuda()
    ref = da @ db.T
    fac, rel = _bound_terms(dt)
    bad = int(((C.double() - ref).abs() > fac * TOL * (da.abs() @ db.abs().T) + ref.abs() * rel).sum())
    assert bad == 0, f"{shape}: {bad} outputs beyond the bound"
    rng = np.random.default_rng(M + fa)
    ms, ns = rng.integers(0, M, 1000), rng.integers(0, N, 1000)
    c64, s = O.gemm_samples(hea, hsa, heb, hsb, M, N, K, fa, fb, ms, ns)
    got = C[torch.from_numpy(ms).cuda(), torch.from_numpy(ns).cuda()].double().cpu().numpy()
    assert (np.abs(got - c64) <= fac * TOL * s + np.abs(c64) * rel).all()


def test_gemm_dense_errors():
    z = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    out = torch.zeros((128, 128), device="cuda")
    with pytest.raises(mx.MxError) as e:
        mx.mx_gemm_dense(z, z, z, z, 128, 128, 128, 5, 5, workspace=z[:1024], out=out)
    assert e.value.status == mx.MX_ERR_WORKSPACE
    with pytest.raises(mx.MxError) as e:
        mx.mx_gemm(z, z, z, z, 128, 128, 128, 5, 0, out=out)
    assert e.value.status == mx.MX_ERR_UNSUPPORTED


@pytest.mark.parametrize("M,N,K,fa,fb,dt", [
    (1, 128, 128, 0, 0, torch.float32),          # a single token
    (7, 4100, 96, 0, 1, torch.float32),          # K tail, N a multiple of 4 only
    (100, 200, 256, 4, 0, torch.bfloat16),       # M and N tails (6- and 4-bit codes: K % 128)
    (300, 37 * 256 + 32, 352, 0, 1, torch.float32),  # 128 x 256 tiles with tails in M, N and K
    (2048, 9608, 416, 1, 1, torch.float32),      # two-CTA tiles, N and K tails
    (2048, 9608, 384, 2, 3, torch.float32),      # 6-bit operands (K % 128)
    (130, 264, 640, 4, 4, torch.bfloat16),
    (640, 4104, 384, 0, 0, torch.float32),       # two-CTA tiles with a half-empty last tile row, N tail
    (900, 8200, 256, 2, 3, torch.bfloat16),      # the same with 6-bit operands and BF16 out
])
def test_tails(M, N, K, fa, fb, dt):
    """Shapes that are not whole tiles: any M, K a multiple of the block size, C rows whole 16-byte
    units.  The copies zero-fill past the edges and the stores are clipped; the guard bands catch a
    store that is not."""
    g = torch.Generator(device="cuda").manual_seed(M + N + K)
    A = torch.randn((M, K), generator=g, device="cuda") * torch.exp(torch.randn((M, 1), generator=g, device="cuda"))
    B = torch.randn((N, K), generator=g, device="cuda") * 0.05
    ea, sa = mx.mx_quantize(A, 1, fa)
    eb, sb = mx.mx_quantize(B, 1, fb)
    esz = 2 if dt == torch.bfloat16 else 4
    g_out = Guarded(M * N * esz)
    C = g_out.view.view(dt).view(M, N)
    if dt == torch.bfloat16:
        mx.mx_gemm_bf16(ea, sa, eb, sb, M, N, K, fa, fb, out=C, check_status=True)
    else:
        mx.mx_gemm(ea, sa, eb, sb, M, N, K, fa, fb, out=C, check_status=True)
    torch.cuda.synchronize()
    g_out.check()
    hea, hsa, heb, hsb = (t.cpu().numpy().reshape(-1) for t in (ea, sa, eb, sb))
    fac, rel = _bound_terms(dt)
    if M * N * K <= 1 << 28:
        c64, s = O.gemm(hea, hsa, heb, hsb, M, N, K, fa, fb)
        got = C.double().cpu().numpy()
    else:
        da = torch.from_numpy(O.dequantize(hea, hsa, M, K, fa, O.F64)).cuda()
        db = torch.from_numpy(O.dequantize(heb, hsb, N, K, fb, O.F64)).cuda()
        ref = da @ db.T
        bad = int(((C.double() - ref).abs() > fac * TOL * (da.abs() @ db.abs().T) + ref.abs() * rel).sum())
        assert bad == 0, f"{bad} outputs beyond the bound"
        rng = np.random.default_rng(K)
        ms = np.concatenate([rng.integers(0, M, 1500), np.full(300, M - 1)])
        ns = np.concatenate([rng.integers(0, N, 1500), rng.integers(N - 40, N, 300)])
        c64, s = O.gemm_samples(hea, hsa, heb, hsb, M, N, K, fa, fb, ms, ns)
        got = C[torch.from_numpy(ms).cuda(), torch.from_numpy(ns).cuda()].double().cpu().numpy()
    assert (np.abs(got - c64) <= fac * TOL * s + np.abs(c64) * rel).all()
    # the BF16 route takes the same shapes
    g_out = Guarded(M * N * esz)
    C2 = g_out.view.view(dt).view(M, N)
    mx.mx_gemm_dense(ea, sa, eb, sb, M, N, K, fa, fb, out=C2, check_status=True)
    torch.cuda.synchronize()
    g_out.check()
    if M * N * K <= 1 << 28:
        assert (np.abs(C2.double().cpu().numpy() - c64) <= fac * TOL * s + np.abs(c64) * rel).all()
    else:
        got2 = C2[torch.from_numpy(ms).cuda(), torch.from_numpy(ns).cuda()].double().cpu().numpy()
        assert (np.abs(got2 - c64) <= fac * TOL * s + np.abs(c64) * rel).all()


def _quantized_operand(x, axis, fmt, rounding, what, seed):
    """Quantizes one GEMM operand on the GPU and proves the bytes before they are used: sampled
    output rows byte for byte against the oracle on the same input, and -- for the transposing
    axis-0 pass, whose kernels are not the last-axis one -- the WHOLE tensor against the last-axis
    kernel run on the transposed input (quantizing along axis 0 is by definition quantizing the
    transpose along its last axis, and that kernel is compared with the oracle on whole tensors)."""
    e, s = mx.mx_quantize(x, axis, fmt, rounding)
    assert_operand_rows_match_oracle(O, x, axis, fmt, rounding, e, s, what, count=256, seed=seed)
    if axis == 0:
        xt = x.t().contiguous()
        e2, s2 = mx.mx_quantize(xt, 1, fmt, rounding)
        assert torch.equal(e, e2) and torch.equal(s, s2), what + ": axis-0 pass differs from the transposed last-axis pass"
        del xt, e2, s2
    return e, s


def test_config3_full_size():
    d = inputs.config3("cuda")
    X, W = d["X"], d["W"]
    M, K = X.shape
    N = W.shape[1]
    ea, sa = _quantized_operand(X, 1, mx.MX_E4M3, mx.MX_RNE, "config 3 X", 31)
    eb, sb = _quantized_operand(W, 0, mx.MX_E4M3, mx.MX_RNE, "config 3 W (axis 0)", 32)
    _full_size_check("config 3", ea, sa, eb, sb, M, N, K, mx.MX_E4M3, mx.MX_E4M3, 3)


def test_config4_training_step():
    """The MXFP6 training step at its own size: FP32 tensors, half-away rounding, every operand
    quantized along its own reduction axis (Section 4.1) and every one of the six compared with
    the oracle before its product is."""
    d = inputs.config4("cuda")
    X, W, dY = d["X"], d["W"], d["dY"]
    n = X.shape[0]
    act, wt, rnd = mx.MX_E3M2, mx.MX_E2M3, mx.MX_RHAZ
    # forward Y = X W: A = Q(X, axis 1), B = Q(W, axis 0) -> [N x K]
    _full_size_check("config 4 fwd", *_quantized_operand(X, 1, act, rnd, "config 4 X rows", 411),
                     *_quantized_operand(W, 0, wt, rnd, "config 4 W columns", 412), n, n, n, act, wt, 41)
    # dgrad dX = dY W^T: A = Q(dY, axis 1), B = Q(W, axis 1)
    _full_size_check("config 4 dgrad", *_quantized_operand(dY, 1, act, rnd, "config 4 dY rows", 421),
                     *_quantized_operand(W, 1, wt, rnd, "config 4 W rows", 422), n, n, n, act, wt, 42)
    # wgrad dW = X^T dY: A = Q(X, axis 0), B = Q(dY, axis 0)
    _full_size_check("config 4 wgrad", *_quantized_operand(X, 0, act, rnd, "config 4 X columns", 431),
                     *_quantized_operand(dY, 0, act, rnd, "config 4 dY columns", 432), n, n, n, act, act, 43)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_config4_dual_axis_operands(dtype):
    """The same six operands out of three mx_quantize_dual calls (each tensor read once): sampled
    rows of both outputs against the oracle, and both outputs whole against the single-axis calls."""
    d = inputs.config4("cuda", dtype=dtype)
    rnd = mx.MX_RHAZ
    for name, fmt in (("X", mx.MX_E3M2), ("W", mx.MX_E2M3), ("dY", mx.MX_E3M2)):
        x = d[name]
        (er, sr), (ec, sc) = mx.mx_quantize_dual(x, fmt, rnd)
        assert_operand_rows_match_oracle(O, x, 1, fmt, rnd, er, sr, f"dual {name} rows", seed=51)
        assert_operand_rows_match_oracle(O, x, 0, fmt, rnd, ec, sc, f"dual {name} columns", seed=52)
        e1, s1 = mx.mx_quantize(x, 1, fmt, rnd)
        e0, s0 = mx.mx_quantize(x, 0, fmt, rnd)
        assert torch.equal(er, e1) and torch.equal(sr, s1), name
        assert torch.equal(ec, e0) and torch.equal(sc, s0), name


def test_config5_full_size():
    d = inputs.config5("cuda")
    W, X = d["W"], d["X"]
    M, K = X.shape
    N = W.shape[1]
    ea, sa = _quantized_operand(X, 1, mx.MX_E4M3, mx.MX_RNE, "config 5 X", 51)
    eb, sb = _quantized_operand(W, 0, mx.MX_E2M1, mx.MX_RNE, "config 5 W (axis 0, FP4)", 52)
    del d, W, X
    torch.cuda.empty_cache()
    _full_size_check("config 5", ea, sa, eb, sb, M, N, K, mx.MX_E4M3, mx.MX_E2M1, 5)


@pytest.mark.parametrize("M,N,K,fa,fb,dt", [
    (4096, 4096, 256, 0, 0, torch.float32),     # 256 tiles on 74 pairs: three whole rounds + 34 tiles in halves
    (2560, 2048, 384, 2, 3, torch.float32),     # 80 tiles: one round + 6 in halves
    (2560, 1984, 512, 4, 4, torch.bfloat16),    # kind::mxf4; the last right halves hold 64 columns
    (2400, 1900, 256, 0, 4, torch.float32),     # ragged in M and N; the last right halves lie past N
    (2304, 4096, 128, 1, 0, torch.bfloat16),    # 144 tiles: one whole round + 70 (more than half the pairs: no halving)
])
def test_last_round_in_halves_equals_whole_tiles(M, N, K, fa, fb, dt):
    """A last round of the two-CTA kernel that would occupy at most half of the CTA pairs is computed
    as items of 128 columns (the library's choice, tile_n = 0).  Whole matrix against the FP64
    product of the oracle-dequantized operands and samples against the oracle, and bit-identical to
    the product computed in whole 256-wide tiles (tile_n = 256)."""
    g = torch.Generator(device="cuda").manual_seed(M + N + K)
    A = torch.randn((M, K), generator=g, device="cuda") * torch.exp(torch.randn((M, 1), generator=g, device="cuda"))
    B = torch.randn((N, K), generator=g, device="cuda") * 0.02
    ea, sa = mx.mx_quantize(A, 1, fa)
    eb, sb = mx.mx_quantize(B, 1, fb)
    esz = 2 if dt == torch.bfloat16 else 4
    g_out = Guarded(M * N * esz)
    C = g_out.view.view(dt).view(M, N)
    mx.mx_gemm_ex(ea, sa, eb, sb, M, N, K, fa, fb, out=C, few_rows_limit=0, check_status=True)
    torch.cuda.synchronize()
    g_out.check()
    hea, hsa, heb, hsb = (t.cpu().numpy().reshape(-1) for t in (ea, sa, eb, sb))
    da = torch.from_numpy(O.dequantize(hea, hsa, M, K, fa, O.F64)).cuda()
    db = torch.from_numpy(O.dequantize(heb, hsb, N, K, fb, O.F64)).cuda()
    ref = da @ db.T
    fac, rel = _bound_terms(dt)
    bad = int(((C.double() - ref).abs() > fac * TOL * (da.abs() @ db.abs().T) + ref.abs() * rel).sum())
    assert bad == 0, f"{bad} outputs beyond the bound"
    rng = np.random.default_rng(K)
    ms = np.concatenate([rng.integers(0, M, 600), np.full(100, M - 1)])
    ns = np.concatenate([rng.integers(0, N, 600), rng.integers(max(0, N - 40), N, 100)])
    c64, s_ = O.gemm_samples(hea, hsa, heb, hsb, M, N, K, fa, fb, ms, ns)
    got = C[torch.from_numpy(ms).cuda(), torch.from_numpy(ns).cuda()].double().cpu().numpy()
    assert (np.abs(got - c64) <= fac * TOL * s_ + np.abs(c64) * rel).all()
    C1 = mx.mx_gemm_ex(ea, sa, eb, sb, M, N, K, fa, fb, out_dtype=dt, tile_n=256, few_rows_limit=0, check_status=True)
    assert torch.equal(C1, C)


@pytest.mark.parametrize("fa,fb,K,dt", [(0, 0, 640, torch.float32), (4, 4, 512, torch.float32), (2, 0, 384, torch.bfloat16)])
def test_wide_tile_variant_whole_matrix(fa, fb, K, dt):
    """The 256 x 384 tile of the two-CTA kernel (mx_gemm_ex, tile_n = 384) on a shape with a ragged
    last tile: whole matrix against the FP64 product of the oracle-dequantized operands, samples
    against the oracle, and bit-identical to the default 256 x 256 tiles."""
    M, N = 2048, 9608
    g = torch.Generator(device="cuda").manual_seed(K + fa)
    A = torch.randn((M, K), generator=g, device="cuda") * torch.exp(torch.randn((M, 1), generator=g, device="cuda"))
    B = torch.randn((N, K), generator=g, device="cuda") * 0.02
    ea, sa = mx.mx_quantize(A, 1, fa)
    eb, sb = mx.mx_quantize(B, 1, fb)
    esz = 2 if dt == torch.bfloat16 else 4
    g_out = Guarded(M * N * esz)
    C = g_out.view.view(dt).view(M, N)
    mx.mx_gemm_ex(ea, sa, eb, sb, M, N, K, fa, fb, out=C, tile_n=384, check_status=True)
    torch.cuda.synchronize()
    g_out.check()
    hea, hsa, heb, hsb = (t.cpu().numpy().reshape(-1) for t in (ea, sa, eb, sb))
    da = torch.from_numpy(O.dequantize(hea, hsa, M, K, fa, O.F64)).cuda()
    db = torch.from_numpy(O.dequantize(heb, hsb, N, K, fb, O.F64)).cuda()
    ref = da @ db.T
    fac, rel = _bound_terms(dt)
    bad = int(((C.double() - ref).abs() > fac * TOL * (da.abs() @ db.abs().T) + ref.abs() * rel).sum())
    assert bad == 0, f"{bad} outputs beyond the bound"
    rng = np.random.default_rng(K)
    ms = np.concatenate([rng.integers(0, M, 1000), np.full(200, M - 1)])
    ns = np.concatenate([rng.integers(0, N, 1000), rng.integers(N - 40, N, 200)])
    c64, s_ = O.gemm_samples(hea, hsa, heb, hsb, M, N, K, fa, fb, ms, ns)
    got = C[torch.from_numpy(ms).cuda(), torch.from_numpy(ns).cuda()].double().cpu().numpy()
    assert (np.abs(got - c64) <= fac * TOL * s_ + np.abs(c64) * rel).all()
    C0 = mx.mx_gemm_ex(ea, sa, eb, sb, M, N, K, fa, fb, out_dtype=dt, check_status=True)   # 256 x 256 tiles
    assert torch.equal(C0, C)


@pytest.mark.parametrize("M,N,K,fa,fb,drop", [
    (256, 256, 1024, 0, 0, 2),     # one-CTA kernel, 128 x 128 tiles
    (1024, 4096, 512, 0, 4, 1),    # two-CTA kernel
    (16, 1024, 1024, 0, 0, 3),     # few rows of A: operands swapped
])
def test_device_wait_runs_out_and_context_survives(M, N, K, fa, fb, drop):
    """Failure detection without a GPU fault: the operand producer is told to leave out one pipeline
    fill (nothing is copied for it, so nothing is in flight later) and every device-side wait gets
    a budget of about a millisecond.  The MMA issuer's wait for that stage must run out, the kernel
    must leave through its common exit (tensor memory released), the checked call must return
    MX_ERR_TIMEOUT naming that wait, and the very next ordinary product on the same context must
    be right against the oracle."""
    g = torch.Generator(device="cuda").manual_seed(M + N + K)
    A = torch.randn((M, K), generator=g, device="cuda")
    B = torch.randn((N, K), generator=g, device="cuda") * 0.1
    ea, sa = mx.mx_quantize(A, 1, fa)
    eb, sb = mx.mx_quantize(B, 1, fb)
    torch.cuda.synchronize()
    with pytest.raises(mx.MxError) as ei:
        mx.mx_gemm_ex(ea, sa, eb, sb, M, N, K, fa, fb, wait_cycles=2_000_000, drop_fill=drop, check_status=True)
    assert ei.value.status == mx.MX_ERR_TIMEOUT
    assert "wait 2 gave up" in str(ei.value), str(ei.value)       # 2 = MMA issuer / stage full
    # the status word was cleared by the failed check; the context and the tensor memory are usable
    g_out = Guarded(M * N * 4)
    C = g_out.view.view(torch.float32).view(M, N)
    mx.mx_gemm(ea, sa, eb, sb, M, N, K, fa, fb, out=C, check_status=True)
    torch.cuda.synchronize()
    g_out.check()
    c64, s_ = O.gemm(*(t.cpu().numpy().reshape(-1) for t in (ea, sa, eb, sb)), M, N, K, fa, fb)
    assert (np.abs(C.double().cpu().numpy() - c64) <= TOL * s_).all()
    # a budget without a drill changes nothing
    C2 = mx.mx_gemm_ex(ea, sa, eb, sb, M, N, K, fa, fb, wait_cycles=2_000_000_000, check_status=True)
    assert torch.equal(C, C2)


def test_host_buffer_gemm():
    M, N, K = 128, 256, 256
    g = torch.Generator(device="cuda").manual_seed(8)
    A = torch.randn((M, K), generator=g, device="cuda")
    B = torch.randn((N, K), generator=g, device="cuda")
    ea, sa = mx.mx_quantize(A, 1, mx.MX_E4M3)
    eb, sb = mx.mx_quantize(B, 1, mx.MX_E2M1)
    ref = mx.mx_gemm(ea, sa, eb, sb, M, N, K, mx.MX_E4M3, mx.MX_E2M1)
    hC = torch.empty((M, N), dtype=torch.float32).pin_memory()
    ws = torch.empty(mx.mx_gemm_host_workspace_bytes(M, N, K, mx.MX_E4M3, mx.MX_E2M1),
                     dtype=torch.uint8, device="cuda")
    mx.mx_gemm_host(ea.cpu().pin_memory(), sa.cpu().pin_memory(), eb.cpu().pin_memory(),
                    sb.cpu().pin_memory(), hC, M, N, K, mx.MX_E4M3, mx.MX_E2M1, ws)
    assert torch.equal(hC, ref.cpu())


def test_output_beyond_4gib():
    """C = 36864 x 36864 FP32 (5.4 GB): output offsets pass 2^32.  Samples from the last rows and
    columns against the oracle; the guard bytes behind the output stay intact."""
    M = N = 36864
    K = 128
    g = torch.Generator(device="cuda").manual_seed(11)
    A = torch.randn((M, K), generator=g, device="cuda")
    B = torch.randn((N, K), generator=g, device="cuda")
    ea, sa = mx.mx_quantize(A, 1, 0)
    eb, sb = mx.mx_quantize(B, 1, 1)
    g_out = Guarded(M * N * 4)
    C = g_out.view.view(torch.float32).view(M, N)
    mx.mx_gemm(ea, sa, eb, sb, M, N, K, 0, 1, out=C, check_status=True)
    torch.cuda.synchronize()
    g_out.check()
    rng = np.random.default_rng(3)
    ms = np.concatenate([rng.integers(0, M, 1500), rng.integers(M - 300, M, 1500), [M - 1, M - 1, 0]])
    ns = np.concatenate([rng.integers(0, N, 1500), rng.integers(N - 300, N, 1500), [N - 1, 0, N - 1]])
    c64, s = O.gemm_samples(*(t.cpu().numpy().reshape(-1) for t in (ea, sa, eb, sb)), M, N, K, 0, 1, ms, ns)
    got = C[torch.from_numpy(ms).cuda(), torch.from_numpy(ns).cuda()].double().cpu().numpy()
    assert (np.abs(got - c64) <= TOL * s).all()
    # every element was written: an untouched output would keep the fill value
    assert not bool((C.view(torch.int32) == -1515870811).any())     # 0xA5A5A5A5


def test_cuda_graph_replay():
    """The device entry points only queue work on the caller's stream, so a step (quantize both
    operands, GEMM, dequantize) can be captured in a CUDA graph after one warm-up call and replayed
    on new data: the replay must give what the eager calls give on that data."""
    M, N, K = 256, 512, 1024
    g = torch.Generator(device="cuda").manual_seed(21)
    A = torch.randn((M, K), generator=g, device="cuda", dtype=torch.bfloat16)
    B = torch.randn((K, N), generator=g, device="cuda", dtype=torch.bfloat16)
    fa, fb = mx.MX_E4M3, mx.MX_E2M1
    ea, sa = mx.mx_quantize(A, 1, fa)
    eb, sb = mx.mx_quantize(B, 0, fb)
    C = torch.empty((M, N), dtype=torch.float32, device="cuda")
    back = torch.empty_like(A)

    def step():
        mx.mx_quantize(A, 1, fa, out=(ea, sa))
        mx.mx_quantize(B, 0, fb, out=(eb, sb))
        mx.mx_gemm(ea, sa, eb, sb, M, N, K, fa, fb, out=C)
        mx.mx_dequantize(ea, sa, [M, K], fa, torch.bfloat16, out=back)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()                      # warm-up: one-time attribute settings happen outside the capture
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    # new data in the same buffers, then replay
    A.copy_(torch.randn((M, K), generator=g, device="cuda").to(torch.bfloat16))
    B.copy_(torch.randn((K, N), generator=g, device="cuda").to(torch.bfloat16) * 0.1)
    graph.replay()
    torch.cuda.synchronize()
    got = (ea.clone(), sa.clone(), eb.clone(), sb.clone(), C.clone(), back.clone())
    step()
    torch.cuda.synchronize()
    for a, b in zip(got, (ea, sa, eb, sb, C, back)):
        assert torch.equal(a.view(torch.uint8), b.view(torch.uint8))
    # and the eager result is the oracle's
    c64, s = O.gemm(*(t.cpu().numpy().reshape(-1) for t in (ea, sa, eb, sb)), M, N, K, fa, fb)
    assert (np.abs(C.double().cpu().numpy() - c64) <= TOL * s).all()
