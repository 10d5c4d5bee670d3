"""GPU parity: mx_quantize / mx_dequantize through the C ABI against the CPU
oracle, byte for byte, on the same seeded inputs."""
import ctypes

import numpy as np
import pytest
import torch

import oracle as O
import paper_2310_10537_b200 as mx
import workloads as inputs
from gpu_util import Guarded, to_oracle_input

pytestmark = pytest.mark.gpu

FMTS = list(range(6))
DTYPES = [torch.float32, torch.bfloat16]


def _quantize_guarded(x, axis, fmt, rounding, layout):
    shape = list(x.shape)
    axis %= len(shape)
    ge = Guarded(mx.mx_elems_bytes(shape, axis, fmt))
    gs = Guarded(mx.mx_scales_bytes(shape, axis, layout))
    mx.mx_quantize(x, axis, fmt, rounding, layout, out=(ge.view, gs.view))
    torch.cuda.synchronize()
    ge.check()
    gs.check()
    return ge.view, gs.view


def _assert_same_bytes(got: torch.Tensor, want: np.ndarray, what):
    got = got.cpu().numpy()
    assert got.shape == want.shape, what
    if not (got == want).all():
        bad = np.flatnonzero(got != want)
        raise AssertionError(f"{what}: {bad.size} bytes differ, first at {bad[0]}: "
                             f"got {got[bad[0]]:#x} want {want[bad[0]]:#x}")


@pytest.mark.parametrize("dtype", DTYPES, ids=["f32", "bf16"])
@pytest.mark.parametrize("fmt", FMTS)
def test_last_axis_adversarial_bit_exact(fmt, dtype):
    # 200 rows x 51 blocks: several CTA tiles, a ragged tail, padding in the swizzled scales
    x = inputs.adversarial("cuda", rows=200, cols=1632, dtype=dtype, seed=11 + fmt)
    xin = to_oracle_input(x)
    for rounding in (mx.MX_RNE, mx.MX_RHAZ):
        for layout in (mx.MX_SCALES_LINEAR, mx.MX_SCALES_SWIZZLED):
            e, s = _quantize_guarded(x, 1, fmt, rounding, layout)
            we, ws = O.quantize(xin, 1, fmt, rounding, layout)
            _assert_same_bytes(e, we, ("elems", fmt, dtype, rounding, layout))
            _assert_same_bytes(s, ws, ("scales", fmt, dtype, rounding, layout))
            e2, s2 = _quantize_guarded(x, 1, fmt, rounding, layout)  # same bytes on a second run
            assert torch.equal(e, e2) and torch.equal(s, s2)


@pytest.mark.parametrize("dtype", DTYPES, ids=["f32", "bf16"])
@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("inner", [1000, 1002, 999])
def test_strided_axis_adversarial_bit_exact(fmt, dtype, inner):
    # blocks along axis 0 of a [352 x inner] tensor (11 blocks deep); inner picks the
    # 4-, 2- or 1-column variant of the kernel
    x = inputs.adversarial("cuda", rows=inner, cols=352, dtype=dtype, seed=5 + fmt).t().contiguous()
    assert list(x.shape) == [352, inner]
    xin = to_oracle_input(x)
    rounding = mx.MX_RHAZ if (fmt + inner) % 2 else mx.MX_RNE
    for layout in (mx.MX_SCALES_LINEAR, mx.MX_SCALES_SWIZZLED):
        e, s = _quantize_guarded(x, 0, fmt, rounding, layout)
        we, ws = O.quantize(xin, 0, fmt, rounding, layout)
        _assert_same_bytes(e, we, ("elems", fmt, dtype, inner, layout))
        _assert_same_bytes(s, ws, ("scales", fmt, dtype, inner, layout))


@pytest.mark.parametrize("dtype", DTYPES, ids=["f32", "bf16"])
@pytest.mark.parametrize("rounding", [mx.MX_RNE, mx.MX_RHAZ])
def test_int8_saturation_boundary(dtype, rounding):
    """MXINT8 saturates at +-127: block maxima that scale to just below, exactly and just above
    127.5 (the smallest value that rounds to 128), of either sign, scattered so that some warps of
    the kernel hold a saturating block and others none (the kernel skips the clamp for those)."""
    rows, cols = 96, 2048
    g = torch.Generator().manual_seed(17)
    x = (torch.rand((rows, cols), generator=g) - 0.5) * 0.5           # |x| < 0.25: never the block maximum
    tops = [127.5 / 64, 127.0 / 64, 1.984375, 1.99609375, 1.0, 127.5 / 64 * 4, -127.5 / 64, -1.99609375 / 8]
    if dtype == torch.float32:
        t = np.float32(127.5 / 64)
        tops += [float(np.nextafter(t, np.float32(0))), float(np.nextafter(t, np.float32(4))),
                 -float(np.nextafter(t, np.float32(0)))]
    k = 0
    for r in range(0, rows, 3):                 # every third row gets maxima, the rows between get none
        for b in range(0, cols // 32, 5):
            x[r, b * 32 + (k * 7) % 32] = tops[k % len(tops)]
            k += 1
    x = x.to(dtype).cuda()
    xin = to_oracle_input(x)
    for layout in (mx.MX_SCALES_LINEAR, mx.MX_SCALES_SWIZZLED):
        e, s = _quantize_guarded(x, 1, mx.MX_INT8, rounding, layout)
        we, ws = O.quantize(xin, 1, mx.MX_INT8, rounding, layout)
        _assert_same_bytes(e, we, ("elems", dtype, rounding, layout))
        _assert_same_bytes(s, ws, ("scales", dtype, rounding, layout))
    assert (we == 0x7F).any() and (we == 0x81).any()   # the clamp did have something to do


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("rows,cols", [(128, 128), (384, 640), (1152, 256)])
def test_strided_axis_whole_tiles_bit_exact(fmt, rows, cols):
    """Axis 0 of 2-D BF16 tensors made of whole 128 x 128 tiles: the shapes from which the 6-bit
    formats take the shared-memory tile kernel's column pass (the others keep the register
    kernels); adversarial blocks, both roundings, both scale layouts, against the oracle."""
    x = inputs.adversarial("cuda", rows=cols, cols=rows, dtype=torch.bfloat16, seed=21 + fmt).t().contiguous()
    assert list(x.shape) == [rows, cols]
    xin = to_oracle_input(x)
    for rounding in (mx.MX_RNE, mx.MX_RHAZ):
        for layout in (mx.MX_SCALES_LINEAR, mx.MX_SCALES_SWIZZLED):
            e, s = _quantize_guarded(x, 0, fmt, rounding, layout)
            we, ws = O.quantize(xin, 0, fmt, rounding, layout)
            _assert_same_bytes(e, we, ("elems", fmt, rows, cols, rounding, layout))
            _assert_same_bytes(s, ws, ("scales", fmt, rows, cols, rounding, layout))


@pytest.mark.parametrize("fmt,rounding", [(mx.MX_E3M2, mx.MX_RNE), (mx.MX_E2M3, mx.MX_RHAZ)])
def test_strided_axis_6bit_at_weight_size(fmt, rounding):
    """The FFN weight of configuration 3 (4096 x 16384 BF16) quantized along axis 0 to the 6-bit
    formats -- the size at which this path is timed, and the one that takes the tile kernel's column
    pass: 256 sampled output rows (both ends, tile seams, middle) byte for byte against the oracle,
    and the whole tensor against the last-axis kernel on the transposed input."""
    from gpu_util import assert_operand_rows_match_oracle
    w = inputs.config3("cuda")["W"]
    assert list(w.shape) == [4096, 16384] and w.dtype == torch.bfloat16
    e, s = mx.mx_quantize(w, 0, fmt, rounding)
    assert_operand_rows_match_oracle(O, w, 0, fmt, rounding, e, s, f"W axis 0 fmt {fmt}", count=256, seed=fmt)
    et, st = mx.mx_quantize(w.t().contiguous(), 1, fmt, rounding)
    assert torch.equal(e, et) and torch.equal(s, st)


@pytest.mark.parametrize("fmt", [mx.MX_E4M3, mx.MX_E3M2, mx.MX_E2M1, mx.MX_INT8])
def test_middle_axis_of_3d_tensor(fmt):
    x = inputs.adversarial("cuda", rows=3 * 40, cols=64, dtype=torch.float32, seed=3)
    x = x.view(3, 40, 64).transpose(1, 2).contiguous()  # [3, 64, 40], blocks along axis 1
    xin = to_oracle_input(x)
    e, s = _quantize_guarded(x, 1, fmt, mx.MX_RNE, mx.MX_SCALES_SWIZZLED)
    we, ws = O.quantize(xin, 1, fmt, mx.MX_RNE, O.SWIZZLED)
    _assert_same_bytes(e, we, "elems")
    _assert_same_bytes(s, ws, "scales")
    # negative axis and a last-axis call on a 3-D tensor
    y = x.transpose(1, 2).contiguous()
    e, s = _quantize_guarded(y, -1, fmt, mx.MX_RHAZ, mx.MX_SCALES_LINEAR)
    we, ws = O.quantize(to_oracle_input(y), 2, fmt, O.RHAZ, O.LINEAR)
    _assert_same_bytes(e, we, "elems")
    _assert_same_bytes(s, ws, "scales")


@pytest.mark.parametrize("dtype,R,C", [(torch.float32, 384, 320), (torch.float32, 256, 384), (torch.float32, 1280, 640),
                                       (torch.bfloat16, 256, 384), (torch.bfloat16, 384, 512),
                                       (torch.bfloat16, 128, 256), (torch.bfloat16, 640, 1280)],
                         ids=["f32", "f32-whole-tiles", "f32-many-tiles", "bf16", "bf16-4-tiles-wide", "bf16-one-row-of-tiles",
                              "bf16-many-tiles"])
@pytest.mark.parametrize("fmt", FMTS)
def test_dual_axis_quantize_matches_both_single_axis_results(fmt, dtype, R, C):
    """mx_quantize_dual reads the tensor once and must write exactly the two tensors that
    quantizing along axis 1 and along axis 0 give (checked against the oracle, not against
    mx_quantize).  BF16 tensors go through the tile kernel (128 x 128 tiles), FP32 tensors through
    the register kernel except 6-bit codes of whole 128 x 128 tiles, which have a tile kernel too."""
    x = inputs.adversarial("cuda", rows=R, cols=C, dtype=dtype, seed=41 + fmt)
    xin = to_oracle_input(x)
    for rounding, layout in ((mx.MX_RNE, mx.MX_SCALES_SWIZZLED), (mx.MX_RHAZ, mx.MX_SCALES_LINEAR)):
        g = [Guarded(mx.mx_elems_bytes([R, C], 1, fmt)), Guarded(mx.mx_scales_bytes([R, C], 1, layout)),
             Guarded(mx.mx_elems_bytes([R, C], 0, fmt)), Guarded(mx.mx_scales_bytes([R, C], 0, layout))]
        # (check_status: the call synchronises and would report a device-side wait that gave up)
        mx.mx_quantize_dual(x, fmt, rounding, layout, out=((g[0].view, g[1].view), (g[2].view, g[3].view)), check_status=True)
        torch.cuda.synchronize()
        for gg in g:
            gg.check()
        wer, wsr = O.quantize(xin, 1, fmt, rounding, layout)
        wec, wsc = O.quantize(xin, 0, fmt, rounding, layout)
        _assert_same_bytes(g[0].view, wer, ("row elems", fmt, dtype, layout))
        _assert_same_bytes(g[1].view, wsr, ("row scales", fmt, dtype, layout))
        _assert_same_bytes(g[2].view, wec, ("col elems", fmt, dtype, layout))
        _assert_same_bytes(g[3].view, wsc, ("col scales", fmt, dtype, layout))
    with pytest.raises(mx.MxError) as ei:
        mx.mx_quantize_dual(torch.zeros((96, 128), dtype=dtype, device="cuda"), fmt)
    assert ei.value.status == mx.MX_ERR_UNSUPPORTED


@pytest.mark.parametrize("fmt", FMTS)
def test_dual_axis_bf16_subnormal_inputs_in_blocks_of_small_maxima(fmt):
    """Algorithm 1 treats FP32-subnormal inputs as zero.  In a block whose maximum is itself tiny the
    scaled value of a subnormal input would reach the element grid if it were not flushed, so the
    kernels may scale BF16 pairs with a packed multiply (which keeps subnormals) only in blocks
    where that cannot happen.  32 x 32 regions with maxima 2^-126 .. 2^-87 (every scale byte from 0
    up past each format's limit), filled with subnormals of both signs, the smallest normals and
    zeros: both outputs byte for byte against the oracle, both roundings."""
    R, C = 256, 256
    g = torch.Generator().manual_seed(7 + fmt)
    bits = torch.randint(0, 0x80, (R, C), generator=g, dtype=torch.int32)          # BF16 subnormals and +0
    bits[torch.rand((R, C), generator=g) < 0.2] = 0x0080                           # smallest normal
    bits |= (torch.randint(0, 2, (R, C), generator=g, dtype=torch.int32) << 15)    # signs
    for i in range(R // 32):
        for j in range(C // 32):
            e = 1 + (i * (C // 32) + j) % 40                                       # biased exponent of the maximum
            r0, c0 = 32 * i, 32 * j
            for d in range(32):                                                    # one per row and per column
                bits[r0 + d, c0 + (5 * d + 3) % 32] = (e << 7) | int(torch.randint(0, 0x80, (1,), generator=g))
    x = bits.to(torch.int16).view(torch.bfloat16).cuda()
    xin = to_oracle_input(x)
    for rounding in (mx.MX_RNE, mx.MX_RHAZ):
        (er, sr), (ec, sc) = mx.mx_quantize_dual(x, fmt, rounding, mx.MX_SCALES_LINEAR)
        wer, wsr = O.quantize(xin, 1, fmt, rounding, O.LINEAR)
        wec, wsc = O.quantize(xin, 0, fmt, rounding, O.LINEAR)
        _assert_same_bytes(er, wer, ("row elems", fmt, rounding))
        _assert_same_bytes(sr, wsr, ("row scales", fmt, rounding))
        _assert_same_bytes(ec, wec, ("col elems", fmt, rounding))
        _assert_same_bytes(sc, wsc, ("col scales", fmt, rounding))
        for axis, (ge, gs) in ((1, (er, sr)), (0, (ec, sc))):                      # and the single-axis kernels
            e1, s1 = mx.mx_quantize(x, axis, fmt, rounding, mx.MX_SCALES_LINEAR)
            assert torch.equal(e1, ge) and torch.equal(s1, gs)


@pytest.mark.parametrize("fmt,rounding,dtype", [(mx.MX_E4M3, mx.MX_RHAZ, torch.bfloat16),
                                                (mx.MX_INT8, mx.MX_RNE, torch.bfloat16),
                                                (mx.MX_E5M2, mx.MX_RNE, torch.float32),
                                                (mx.MX_E3M2, mx.MX_RHAZ, torch.float32)])
def test_dual_axis_at_sweep_size(fmt, rounding, dtype):
    """The 8192 x 8192 sweep tensor through mx_quantize_dual (the size it is timed at; BF16 with 8-bit
    codes takes the kernel with 128 x 256 tiles, FP32 with 8-bit codes the register kernel in its
    many-waves configuration, FP32 with 6-bit codes its staged form): 256 sampled rows of each of the
    two outputs byte for byte against the oracle, and both whole tensors against the single-axis
    kernels."""
    from gpu_util import assert_operand_rows_match_oracle
    x = inputs.config2("cuda")
    assert list(x.shape) == [8192, 8192] and x.dtype == torch.bfloat16
    x = x.to(dtype)
    (er, sr), (ec, sc) = mx.mx_quantize_dual(x, fmt, rounding)
    assert_operand_rows_match_oracle(O, x, 1, fmt, rounding, er, sr, "dual, row blocks", count=256, seed=1)
    assert_operand_rows_match_oracle(O, x, 0, fmt, rounding, ec, sc, "dual, column blocks", count=256, seed=2)
    e1, s1 = mx.mx_quantize(x, 1, fmt, rounding)
    e0, s0 = mx.mx_quantize(x, 0, fmt, rounding)
    assert torch.equal(er, e1) and torch.equal(sr, s1) and torch.equal(ec, e0) and torch.equal(sc, s0)


def test_dual_axis_many_launches_on_two_streams():
    """The tile kernels of mx_quantize_dual deal their tiles out at run time from per-launch counter
    slots that the host hands out round-robin (256 of them) and the kernels leave at zero.  More
    launches than slots, interleaved on two streams with different shapes, formats and input types:
    every result equals the single-axis kernels' (which the other tests pin to the oracle)."""
    cases = [(torch.bfloat16, 512, 1024, mx.MX_E4M3), (torch.bfloat16, 1280, 384, mx.MX_E2M1),
             (torch.bfloat16, 256, 2048, mx.MX_E3M2), (torch.float32, 640, 768, mx.MX_E2M3)]
    g = torch.Generator(device="cuda").manual_seed(99)
    xs, want = [], []
    for dt, R, C, fmt in cases:
        x = (torch.randn((R, C), generator=g, device="cuda") * torch.exp(torch.randn((R, 1), generator=g, device="cuda"))).to(dt)
        xs.append(x)
        want.append((mx.mx_quantize(x, 1, fmt), mx.mx_quantize(x, 0, fmt)))
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = [[mx.mx_quantize_dual(x, fmt) for (_, _, _, fmt), x in zip(cases, xs)] for _ in streams]
    torch.cuda.synchronize()
    for rep in range(90):                       # 90 x 4 cases x 2 streams = 720 launches
        for si, st in enumerate(streams):
            with torch.cuda.stream(st):
                for ci, ((_, _, _, fmt), x) in enumerate(zip(cases, xs)):
                    if rep % 30 == 29:          # poison the outputs now and then, so stale results cannot pass
                        for pair in outs[si][ci]:
                            for t in pair:
                                t.fill_(0xA5)
                    mx.mx_quantize_dual(x, fmt, out=outs[si][ci])
    torch.cuda.synchronize()
    for si in range(2):
        for ci in range(len(cases)):
            (er, sr), (ec, sc) = outs[si][ci]
            (e1, s1), (e0, s0) = want[ci]
            assert torch.equal(er, e1) and torch.equal(sr, s1) and torch.equal(ec, e0) and torch.equal(sc, s0), (si, ci)


def test_worked_blocks_on_device():
    """The hand-worked W1 / W4 / W5 blocks straight through the kernel."""
    v = torch.zeros(32, device="cuda")
    v[:6] = torch.tensor([100, 1, -0.75, 0.3, 0.001, -1e-30])
    e, s = mx.mx_quantize(v.view(1, 32), 1, mx.MX_E4M3, mx.MX_RNE, mx.MX_SCALES_LINEAR)
    assert e[:6].tolist() == [0x7C, 0x48, 0xC4, 0x3A, 0x02, 0x80] and s.tolist() == [0x7D]
    e, s = mx.mx_quantize(v.view(1, 32), 1, mx.MX_E4M3, mx.MX_RHAZ, mx.MX_SCALES_LINEAR)
    assert e[0].item() == 0x7D
    w4 = [6, 5, 4, 3.5, 3, 2.5, 2, 1.75, 1.5, 1.25, 1, 0.75, 0.5, 0.25, 0.2, 0, -0.25, -6, 7]
    v = torch.zeros(32, device="cuda")
    v[:len(w4)] = torch.tensor(w4)
    e, s = mx.mx_quantize(v.view(1, 32), 1, mx.MX_E2M1, mx.MX_RNE, mx.MX_SCALES_LINEAR)
    assert e[:10].tolist() == [0x67, 0x66, 0x45, 0x44, 0x23, 0x22, 0x01, 0x00, 0xF8, 0x07]
    assert s.tolist() == [0x7F]
    v = torch.zeros(32, device="cuda")
    v[:7] = torch.tensor([1.5, -1.5, 1.9921875, 0.0078125, -0.0078125, 0.0234375, 1])
    e, _ = mx.mx_quantize(v.view(1, 32), 1, mx.MX_INT8, mx.MX_RHAZ, mx.MX_SCALES_LINEAR)
    assert e[:7].tolist() == [0x60, 0xA0, 0x7F, 0x01, 0xFF, 0x02, 0x40]
    # FP6 bit order: codes 1..8 of E2M3 are the values 0.125 .. 1.0
    v = torch.zeros(32, device="cuda")
    v[:8] = torch.arange(1, 9, device="cuda") * 0.125
    v[31] = 4.0  # pins the scale at 2^0
    e, s = mx.mx_quantize(v.view(1, 32), 1, mx.MX_E2M3, mx.MX_RNE, mx.MX_SCALES_LINEAR)
    assert s.tolist() == [0x7F] and e[:6].tolist() == [0x81, 0x30, 0x10, 0x85, 0x71, 0x20]


@pytest.mark.parametrize("dtype", DTYPES, ids=["f32", "bf16"])
@pytest.mark.parametrize("fmt", FMTS)
def test_dequantize_every_code_and_scale(fmt, dtype):
    rows, L = 130, 32 * 37
    rng = np.random.default_rng(100 + fmt)
    nbytes = rows * L * O.fmt_bits(fmt) // 8
    elems = rng.integers(0, 256, nbytes, dtype=np.uint8)
    out_dt = O.BF16 if dtype == torch.bfloat16 else O.F32
    for layout in (O.LINEAR, O.SWIZZLED):
        scales = rng.integers(0, 256, O.scales_bytes(rows, L // 32, layout), dtype=np.uint8)
        scales[:64] = np.tile(np.array([0, 1, 254, 255, 127, 2, 253, 126], np.uint8), 8)
        want = O.dequantize(elems, scales, rows, L, fmt, out_dt, layout)
        g = Guarded(rows * L * (2 if dtype == torch.bfloat16 else 4))
        out = g.view.view(dtype).view(rows, L)
        mx.mx_dequantize(torch.from_numpy(elems).cuda(), torch.from_numpy(scales).cuda(),
                         [rows, L], fmt, dtype, layout, out=out)
        torch.cuda.synchronize()
        g.check()
        if dtype == torch.bfloat16:
            got = out.view(torch.int16).cpu().numpy().view(np.uint16)
        else:
            got = out.view(torch.int32).cpu().numpy().view(np.uint32)
            want = want.view(np.uint32)
        assert (got == want).all(), (fmt, dtype, layout, int((got != want).sum()))


@pytest.mark.parametrize("fmt", FMTS)
def test_quantize_dequantize_round_trip_is_fixed_point(fmt):
    x = inputs.adversarial("cuda", rows=64, cols=512, dtype=torch.float32, seed=77, nonfinite=False)
    e, s = mx.mx_quantize(x, 1, fmt, layout=mx.MX_SCALES_LINEAR)
    d = mx.mx_dequantize(e, s, [64, 512], fmt, torch.float32, mx.MX_SCALES_LINEAR)
    e2, s2 = mx.mx_quantize(d, 1, fmt, layout=mx.MX_SCALES_LINEAR)
    # Q(D(Q(V))) == Q(V) for every block whose elements all dequantize to normal FP32
    # numbers (with a scale near 2^-127 they become FP32 subnormals, which Algorithm 1 flushes)
    keep = s >= 32
    assert int(keep.sum()) > 500
    assert torch.equal(s[keep], s2[keep])
    bpb = 32 * mx.mx_fmt_bits(fmt) // 8
    assert torch.equal(e.view(-1, bpb)[keep], e2.view(-1, bpb)[keep])


def test_empty_and_error_paths_on_device():
    x = torch.empty((0, 64), device="cuda")
    e, s = mx.mx_quantize(x, 1, mx.MX_E4M3)
    assert e.numel() == 0 and s.numel() == 0
    shape_neg = (ctypes.c_int64 * 2)(4, -48)
    z = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    assert mx.lib().mx_quantize(z.data_ptr(), z.data_ptr() + 1024, z.data_ptr() + 2048, shape_neg, 2, 1, 0, 0,
                                None) == mx.MX_ERR_SHAPE
    buf = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    shape = (ctypes.c_int64 * 2)(4, 64)
    rc = mx.lib().mx_quantize(buf.data_ptr() + 4, buf.data_ptr() + 2048, buf.data_ptr() + 3072,
                              shape, 2, 1, 0, 0, None)
    assert rc == mx.MX_ERR_ALIGN


def test_host_buffer_entry_points():
    x = inputs.adversarial("cpu", rows=64, cols=256, dtype=torch.bfloat16, seed=2).pin_memory()
    shape = [64, 256]
    for fmt in (mx.MX_E4M3, mx.MX_E2M3, mx.MX_E2M1):
        elems = torch.empty(mx.mx_elems_bytes(shape, 1, fmt), dtype=torch.uint8).pin_memory()
        scales = torch.empty(mx.mx_scales_bytes(shape, 1), dtype=torch.uint8).pin_memory()
        ws = torch.empty(mx.mx_quantize_host_workspace_bytes(shape, 1, fmt, torch.bfloat16),
                         dtype=torch.uint8, device="cuda")
        mx.mx_quantize_host(x, elems, scales, 1, fmt, mx.MX_RNE, ws)
        we, ws_ = O.quantize(to_oracle_input(x), 1, fmt, O.RNE, O.SWIZZLED)
        assert (elems.numpy() == we).all() and (scales.numpy() == ws_).all()
        out = torch.empty(shape, dtype=torch.bfloat16).pin_memory()
        ws2 = torch.empty(mx.mx_dequantize_host_workspace_bytes(shape, fmt, torch.bfloat16),
                          dtype=torch.uint8, device="cuda")
        mx.mx_dequantize_host(elems, scales, out, fmt, ws2)
        want = O.dequantize(we, ws_, 64, 256, fmt, O.BF16, O.SWIZZLED)
        assert (out.view(torch.int16).numpy().view(np.uint16) == want).all()
        with pytest.raises(mx.MxError) as ei:
            mx.mx_quantize_host(x, elems, scales, 1, fmt, mx.MX_RNE, ws[:256])
        assert ei.value.status == mx.MX_ERR_WORKSPACE


@pytest.mark.parametrize("rows,cols,dtype,fmt,layout", [
    (2048, 4096, torch.bfloat16, 0, 1),     # eight chunks of 256 rows
    (1000, 4064, torch.float32, 2, 1),      # ragged: last chunk of 104 rows, 127 blocks per row (padded chunks)
    (1000, 4064, torch.float32, 4, 0),      # the same with linear scales
    (700, 8192, torch.bfloat16, 5, 1),
    (600, 4100, torch.float32, 3, 1),       # a partial last block in every row, chunked
    (50, 70, torch.bfloat16, 0, 0),         # the same below the chunking limit
])
def test_host_buffer_entry_points_pipelined(rows, cols, dtype, fmt, layout):
    """Sizes at which the host-buffer calls cut the tensor into row chunks and overlap the copies
    of neighbouring chunks on two internal streams: every output byte against the oracle, guard
    bytes around the pinned outputs intact."""
    padded = (cols + 31) // 32 * 32      # the generator builds whole blocks; a tail is cut afterwards
    x = inputs.adversarial("cpu", rows=rows, cols=padded, dtype=dtype, seed=rows + fmt)[:, :cols].contiguous().pin_memory()
    shape = [rows, cols]
    G = 4096
    eb, sb = mx.mx_elems_bytes(shape, 1, fmt), mx.mx_scales_bytes(shape, 1, layout)
    e_raw = torch.full((eb + 2 * G,), 0xA5, dtype=torch.uint8).pin_memory()
    s_raw = torch.full((sb + 2 * G,), 0xA5, dtype=torch.uint8).pin_memory()
    elems, scales = e_raw[G:G + eb], s_raw[G:G + sb]
    ws = torch.empty(mx.mx_quantize_host_workspace_bytes(shape, 1, fmt, dtype, layout), dtype=torch.uint8, device="cuda")
    mx.mx_quantize_host(x, elems, scales, 1, fmt, mx.MX_RHAZ, ws, layout)
    we, ws_ = O.quantize(to_oracle_input(x), 1, fmt, O.RHAZ, layout)
    assert (elems.numpy() == we).all() and (scales.numpy() == ws_).all()
    for raw, n in ((e_raw, eb), (s_raw, sb)):
        assert bool((raw[:G] == 0xA5).all()) and bool((raw[G + n:] == 0xA5).all())
    o_raw = torch.full((rows * cols * x.element_size() + 2 * G,), 0xA5, dtype=torch.uint8).pin_memory()
    out = o_raw[G:G + rows * cols * x.element_size()].view(dtype).view(rows, cols)
    ws2 = torch.empty(mx.mx_dequantize_host_workspace_bytes(shape, fmt, dtype, layout), dtype=torch.uint8, device="cuda")
    mx.mx_dequantize_host(elems, scales, out, fmt, ws2, layout)
    want = O.dequantize(we, ws_, rows, cols, fmt, O.BF16 if dtype == torch.bfloat16 else O.F32, layout)
    got = out.view(torch.int16).numpy().view(np.uint16) if dtype == torch.bfloat16 else out.numpy()
    assert np.array_equal(got.view(np.uint8), want.view(np.uint8))
    assert bool((o_raw[:G] == 0xA5).all()) and bool((o_raw[-G:] == 0xA5).all())


@pytest.mark.parametrize("fmt", FMTS)
def test_config2_full_size_sweep(fmt):
    """The 8192 x 8192 BF16 sweep tensor in the launch configuration the benchmark
    times: quantize, then dequantize back to BF16.  E4M3 is compared on the whole
    tensor, the other formats on 512 sampled rows (rows are independent)."""
    T = inputs.config2("cuda")
    rows, cols = T.shape
    if fmt == mx.MX_E4M3:
        sel = np.arange(rows)
    else:
        sel = np.sort(np.random.default_rng(fmt).choice(rows, 512, replace=False))
    sel_t = torch.from_numpy(sel).cuda()
    Tin = to_oracle_input(T[sel_t].contiguous())
    w = O.fmt_bits(fmt)
    for rounding in (mx.MX_RNE, mx.MX_RHAZ):
        e, s = mx.mx_quantize(T, 1, fmt, rounding, mx.MX_SCALES_LINEAR)
        d = mx.mx_dequantize(e, s, [rows, cols], fmt, torch.bfloat16, mx.MX_SCALES_LINEAR)
        we, ws = O.quantize(Tin, 1, fmt, rounding, O.LINEAR)
        ge = e.view(rows, cols * w // 8)[sel_t].cpu().numpy().reshape(-1)
        gs = s.view(rows, cols // 32)[sel_t].cpu().numpy().reshape(-1)
        assert (ge == we).all() and (gs == ws).all(), (fmt, rounding)
        wd = O.dequantize(we, ws, sel.size, cols, fmt, O.BF16, O.LINEAR)
        gd = d[sel_t].view(torch.int16).cpu().numpy().view(np.uint16)
        assert (gd == wd).all(), (fmt, rounding)
        if rounding == mx.MX_RNE:
            # swizzled scales hold the same bytes in the other order
            e2, s2 = mx.mx_quantize(T, 1, fmt, rounding, mx.MX_SCALES_SWIZZLED)
            assert torch.equal(e, e2)
            r = torch.arange(rows, device="cuda").view(-1, 1)
            k = torch.arange(cols // 32, device="cuda").view(1, -1)
            off = ((r // 128) * ((cols // 32 + 3) // 4) + k // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + k % 4
            assert torch.equal(s2[off.reshape(-1)], s)
    # structure of the workload: the zero and tiny blocks are really there
    if fmt == mx.MX_E4M3:
        sb = s.cpu().numpy()
        assert 0.0005 < (sb == 0).mean() < 0.002
        assert 0.0005 < ((sb > 0) & (sb < 40)).mean() < 0.002


def test_offsets_beyond_4gib():
    """A 6.4 GB BF16 tensor (49152 x 65536): byte offsets of input, codes and outputs pass 2^32.
    Sampled rows from both ends and the middle against the oracle, last axis and strided axis,
    and the dequantized tensor."""
    rows, cols = 49152, 65536
    g = torch.Generator(device="cuda").manual_seed(99)
    x = torch.empty((rows, cols), dtype=torch.bfloat16, device="cuda")
    for r0 in range(0, rows, 8192):   # filled in slabs: no FP32 copy of the whole tensor
        x[r0:r0 + 8192] = (torch.randn((8192, cols), generator=g, device="cuda") *
                           torch.exp(torch.randn((8192, 1), generator=g, device="cuda"))).to(torch.bfloat16)
    sel = np.array([0, 1, 127, 128, 20000, 32767, 32768, 32769, 40001, rows - 129, rows - 2, rows - 1])
    sel_t = torch.from_numpy(sel).cuda()
    xin = to_oracle_input(x[sel_t].contiguous())
    for fmt in (mx.MX_E4M3, mx.MX_E3M2):
        w = O.fmt_bits(fmt)
        e, s = mx.mx_quantize(x, 1, fmt, mx.MX_RNE, mx.MX_SCALES_LINEAR)
        we, ws = O.quantize(xin, 1, fmt, O.RNE, O.LINEAR)
        assert np.array_equal(e.view(rows, cols * w // 8)[sel_t].cpu().numpy().reshape(-1), we)
        assert np.array_equal(s.view(rows, cols // 32)[sel_t].cpu().numpy().reshape(-1), ws)
        d = mx.mx_dequantize(e, s, [rows, cols], fmt, torch.bfloat16, mx.MX_SCALES_LINEAR)
        want = O.dequantize(we, ws, len(sel), cols, fmt, O.BF16, O.LINEAR)
        assert np.array_equal(d[sel_t].view(torch.int16).cpu().numpy().view(np.uint16), want)
        del e, s, d
    # blocks along axis 0: output row = input column; columns from both ends
    csel = np.array([0, 3, 4, 31, 32768, cols - 5, cols - 1])
    csel_t = torch.from_numpy(csel).cuda()
    e, s = mx.mx_quantize(x, 0, mx.MX_E4M3, mx.MX_RHAZ, mx.MX_SCALES_LINEAR)
    xt = to_oracle_input(x[:, csel_t].t().contiguous())           # [columns, rows]: blocks along the last axis
    we, ws = O.quantize(xt, 1, mx.MX_E4M3, O.RHAZ, O.LINEAR)
    assert np.array_equal(e.view(cols, rows)[csel_t].cpu().numpy().reshape(-1), we)
    assert np.array_equal(s.view(cols, rows // 32)[csel_t].cpu().numpy().reshape(-1), ws)


def test_queued_host_calls():
    """Six quantizes queued back to back (own outputs and workspaces), one synchronize, then six
    queued dequantizes: every byte against the oracle.  Sizes on both sides of the chunking limit."""
    for rows, cols in ((2048, 4096), (96, 512)):
        x = inputs.adversarial("cpu", rows=rows, cols=cols, dtype=torch.bfloat16, seed=rows).pin_memory()
        shape = [rows, cols]
        outs, wss = [], []
        for fmt in FMTS:
            e = torch.full((mx.mx_elems_bytes(shape, 1, fmt),), 0xA5, dtype=torch.uint8).pin_memory()
            s = torch.full((mx.mx_scales_bytes(shape, 1),), 0xA5, dtype=torch.uint8).pin_memory()
            ws = torch.empty(mx.mx_quantize_host_workspace_bytes(shape, 1, fmt, torch.bfloat16), dtype=torch.uint8, device="cuda")
            outs.append((e, s))
            wss.append(ws)
            mx.mx_quantize_host(x, e, s, 1, fmt, mx.MX_RNE, ws, queue=True)
        mx.mx_host_synchronize()
        want = []
        for fmt, (e, s) in zip(FMTS, outs):
            we, ws_ = O.quantize(to_oracle_input(x), 1, fmt, O.RNE, O.SWIZZLED)
            assert (e.numpy() == we).all() and (s.numpy() == ws_).all(), fmt
            want.append(O.dequantize(we, ws_, rows, cols, fmt, O.BF16, O.SWIZZLED))
        backs = []
        for fmt, (e, s), ws in zip(FMTS, outs, wss):
            out = torch.zeros(shape, dtype=torch.bfloat16).pin_memory()
            backs.append(out)
            mx.mx_dequantize_host(e, s, out, fmt, ws, queue=True)
        mx.mx_host_synchronize()
        for fmt, out, w in zip(FMTS, backs, want):
            assert (out.view(torch.int16).numpy().view(np.uint16) == w).all(), fmt


@pytest.mark.parametrize("shape,axis", [
    ((5, 40), 1), ((300, 1), 1), ((129, 31), 1), ((7, 100), 1), ((64, 4100), 1),      # last axis
    ((40, 300), 0), ((33, 7), 0), ((100, 130), 0), ((1, 257), 0),                    # strided axis
    ((3, 50, 6), 1), ((2, 3, 45), 2),
])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_partial_blocks(shape, axis, dtype):
    """Axis lengths that are not multiples of 32: a partial last block, rows stored padded with zero
    codes.  Codes, scales and the dequantized tensor byte for byte against the oracle, six formats,
    both layouts, guard bands around the outputs."""
    g = torch.Generator(device="cuda").manual_seed(sum(shape) + axis)
    x = (torch.randn(shape, generator=g, device="cuda") * torch.exp(2 * torch.randn(shape[:1] + (1,) * (len(shape) - 1), generator=g, device="cuda"))).to(dtype)
    x.view(-1)[::17] = 0.0
    x.view(-1)[3::29] = float("inf") if x.numel() > 40 else 1.0
    L = shape[axis]
    rows = x.numel() // L
    for fmt in FMTS:
        for layout in (mx.MX_SCALES_LINEAR, mx.MX_SCALES_SWIZZLED):
            nb_e, nb_s = mx.mx_elems_bytes(list(shape), axis, fmt), mx.mx_scales_bytes(list(shape), axis, layout)
            ge, gs = Guarded(nb_e), Guarded(nb_s)
            mx.mx_quantize(x, axis, fmt, mx.MX_RHAZ, layout, out=(ge.view, gs.view))
            torch.cuda.synchronize()
            ge.check()
            gs.check()
            we, ws = O.quantize(to_oracle_input(x), axis, fmt, O.RHAZ, layout)
            assert nb_e == we.size and nb_s == ws.size
            assert np.array_equal(ge.view.cpu().numpy(), we), (fmt, layout, "codes")
            assert np.array_equal(gs.view.cpu().numpy(), ws), (fmt, layout, "scales")
            # back: the packed tensor is [rows, L] with blocks along its last axis
            go = Guarded(rows * L * x.element_size())
            out = go.view.view(dtype).view(rows, L)
            mx.mx_dequantize(ge.view, gs.view, [rows, L], fmt, dtype, layout, out=out)
            torch.cuda.synchronize()
            go.check()
            want = O.dequantize(we, ws, rows, L, fmt, O.BF16 if dtype == torch.bfloat16 else O.F32, layout)
            got = out.view(torch.int16).cpu().numpy().view(np.uint16) if dtype == torch.bfloat16 else out.cpu().numpy()
            assert np.array_equal(got.view(np.uint8), want.view(np.uint8)), (fmt, layout, "dequantized")


def test_partial_block_operand_feeds_the_gemm():
    """A K that is not a multiple of 32: the padded rows are a valid operand with K rounded up."""
    M, N, K = 256, 384, 200
    Kp = 224
    g = torch.Generator(device="cuda").manual_seed(5)
    A = torch.randn((M, K), generator=g, device="cuda")
    B = torch.randn((N, K), generator=g, device="cuda")
    ea, sa = mx.mx_quantize(A, 1, mx.MX_E4M3)
    eb, sb = mx.mx_quantize(B, 1, mx.MX_E5M2)
    C = mx.mx_gemm(ea, sa, eb, sb, M, N, Kp, mx.MX_E4M3, mx.MX_E5M2, check_status=True)
    oa, osa = O.quantize(A.cpu().numpy(), 1, O.E4M3)
    ob, osb = O.quantize(B.cpu().numpy(), 1, O.E5M2)
    c64, s = O.gemm(oa, osa, ob, osb, M, N, Kp, O.E4M3, O.E5M2)
    assert (np.abs(C.double().cpu().numpy() - c64) <= 1e-5 * s).all()
