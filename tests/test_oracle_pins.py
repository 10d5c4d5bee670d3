"""Pins for the CPU oracle: everything here checks ``oracle/`` against something
other than itself -- hand-worked blocks, library conversions (ml_dtypes), brute
force over every code of the small formats, closed forms and invariants that
follow from Algorithm 1 (Section 3) and the value rule of Section 2."""
import itertools
import os

import ml_dtypes
import numpy as np
import pytest

import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_blocks.txt")
FMTS = [O.E4M3, O.E5M2, O.E3M2, O.E2M3, O.E2M1, O.INT8]
FP_FMTS = FMTS[:5]
ML = {O.E4M3: ml_dtypes.float8_e4m3fn, O.E5M2: ml_dtypes.float8_e5m2,
      O.E3M2: ml_dtypes.float6_e3m2fn, O.E2M3: ml_dtypes.float6_e2m3fn,
      O.E2M1: ml_dtypes.float4_e2m1fn}
# Table 1 formats: (bits, emax_elem, largest normal) as the OCP specs give them.
PARAMS = {O.E4M3: (8, 8, 448.0), O.E5M2: (8, 15, 57344.0), O.E3M2: (6, 4, 28.0),
          O.E2M3: (6, 2, 7.5), O.E2M1: (4, 2, 6.0), O.INT8: (8, 0, 127 / 64)}


def _eval_num(tok):
    allowed = set("0123456789.e+-* ")
    assert set(tok) <= allowed, tok
    return np.float32(eval(tok, {"__builtins__": {}}, {}))


def _cases():
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            cid, fmt, inputs, scale, rne, rhaz = [p.strip() for p in line.split(";")]
            vals = [_eval_num(t) for t in inputs.split()]
            rne_c = [int(t, 16) for t in rne.split()]
            rhaz_c = rne_c if rhaz == "=" else [int(t, 16) for t in rhaz.split()]
            yield cid, O.FORMATS[fmt], vals, int(scale, 16), rne_c, rhaz_c


@pytest.mark.parametrize("case", list(_cases()), ids=lambda c: c[0])
def test_hand_worked_blocks(case):
    cid, fmt, vals, scale, rne_c, rhaz_c = case
    v = np.zeros(32, dtype=np.float32)
    v[:len(vals)] = vals
    for mode, want in ((O.RNE, rne_c), (O.RHAZ, rhaz_c)):
        codes, sb = O.quantize_block(v, fmt, mode)
        assert sb == scale, (cid, mode, hex(sb))
        assert list(codes[:len(want)]) == want, (cid, mode, [hex(c) for c in codes[:len(want)]])
        assert not codes[len(want):].any()


def test_w4_packed_bytes_and_fp6_pack_pattern():
    # FP4: element 2j in the low nibble of byte j (little-endian bit stream)
    v = np.zeros(32, dtype=np.float32)
    w4 = [6, 5, 4, 3.5, 3, 2.5, 2, 1.75, 1.5, 1.25, 1, 0.75, 0.5, 0.25, 0.2, 0, -0.25, -6, 7]
    v[:len(w4)] = w4
    e, s = O.quantize(v.reshape(1, 32), 1, O.E2M1, O.RNE, O.LINEAR)
    assert list(e[:10]) == [0x67, 0x66, 0x45, 0x44, 0x23, 0x22, 0x01, 0x00, 0xF8, 0x07]
    assert list(s) == [0x7F]
    # FP6: 4 codes in 3 bytes, code i at bits [6i, 6i+6)
    assert list(O.pack_codes(np.array([0x1C, 0x18, 0x3F, 0x01], np.uint8), O.E3M2)) == [0x1C, 0xF6, 0x07]
    assert list(O.pack_codes(np.arange(1, 9, dtype=np.uint8), O.E2M3)) == [0x81, 0x30, 0x10, 0x85, 0x71, 0x20]
    rng = np.random.default_rng(0)
    for fmt in FMTS:
        bits = PARAMS[fmt][0]
        codes = rng.integers(0, 1 << bits, 96, dtype=np.uint8)
        assert (O.unpack_codes(O.pack_codes(codes, fmt), 96, fmt) == codes).all()


def test_format_parameters_match_table():
    for fmt in FMTS:
        bits, emax, mx = PARAMS[fmt]
        assert O.fmt_bits(fmt) == bits
        assert O.fmt_emax(fmt) == emax
        assert O.fmt_max_normal(fmt) == mx
    for fmt in FP_FMTS:
        fi = ml_dtypes.finfo(ML[fmt])
        assert float(fi.max) == PARAMS[fmt][2]
        assert int(np.floor(np.log2(float(fi.max)))) == PARAMS[fmt][1]


@pytest.mark.parametrize("fmt", FP_FMTS)
def test_decode_table_matches_ml_dtypes(fmt):
    bits = PARAMS[fmt][0]
    codes = np.arange(1 << bits, dtype=np.uint8)
    lib_vals = codes.view(ML[fmt]).astype(np.float32) if bits == 8 else None
    if lib_vals is None:
        # sub-byte ml_dtypes types store one code per byte
        lib_vals = codes.view(ML[fmt]).astype(np.float32)
    for c in codes:
        mine = O.decode_element(int(c), fmt)
        ref = float(lib_vals[c])
        if np.isnan(ref):
            assert np.isnan(mine), (fmt, c)
        else:
            assert mine == ref and np.signbit(mine) == np.signbit(ref), (fmt, c, mine, ref)


def test_decode_special_codes_and_int8():
    assert np.isnan(O.decode_element(0x7F, O.E4M3)) and np.isnan(O.decode_element(0xFF, O.E4M3))
    assert O.decode_element(0x7E, O.E4M3) == 448.0
    assert O.decode_element(0x7C, O.E5M2) == np.inf and O.decode_element(0xFC, O.E5M2) == -np.inf
    for c in (0x7D, 0x7E, 0x7F, 0xFD, 0xFE, 0xFF):
        assert np.isnan(O.decode_element(c, O.E5M2))
    for c in range(256):
        assert O.decode_element(c, O.INT8) == np.int8(np.uint8(c)) / 64.0
    assert O.decode_element(0x80, O.INT8) == -2.0


def _finite_grid(fmt):
    """All finite magnitudes of a format with their codes, from the decode table."""
    bits = PARAMS[fmt][0]
    out = []
    for c in range(1 << (bits - 1)) if fmt != O.INT8 else range(128):
        v = O.decode_element(c, fmt)
        if np.isfinite(v):
            out.append((v, c))
    out.sort()
    return out


def _nearest_brute(r, fmt, mode):
    """Definition of rounding by brute force over every code: nearest finite
    grid value (saturating), ties by the mode."""
    grid = _finite_grid(fmt)
    a = abs(r)
    best = None
    for v, c in grid:
        d = abs(v - a)
        if best is None or d < best[0]:
            best = (d, v, c)
        elif d == best[0]:
            if mode == O.RHAZ:
                best = (d, v, c)  # grid is ascending: the later one is larger
            else:
                # ties to even: even mantissa lsb (even code for FP, even n for INT8)
                if c % 2 == 0:
                    best = (d, v, c)
    return best[2]


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("mode", [O.RNE, O.RHAZ])
def test_encode_against_brute_force_nearest(fmt, mode):
    grid = _finite_grid(fmt)
    vals = [v for v, _ in grid]
    probes = []
    for lo, hi in zip(vals[:-1], vals[1:]):
        mid = (lo + hi) / 2
        probes += [lo, mid, np.nextafter(np.float32(mid), np.float32(0)),
                   np.nextafter(np.float32(mid), np.float32(1e9)), hi]
        probes += list(np.linspace(lo, hi, 7)[1:-1])
    top = vals[-1]
    probes += [top, top * 1.01, top * 1.5, 2.0 ** (PARAMS[fmt][1] + 1) * (1 - 2.0 ** -20), vals[1] / 4, vals[1] / 2]
    signbit_shift = PARAMS[fmt][0] - 1
    for r in probes:
        r = float(np.float32(r))
        want = _nearest_brute(r, fmt, mode)
        assert O.encode_element(r, fmt, mode) == want, (fmt, mode, r)
        neg = O.encode_element(-r, fmt, mode)
        if fmt == O.INT8:
            assert neg == (-want) & 0xFF
        else:
            assert neg == want | (1 << signbit_shift)


@pytest.mark.parametrize("fmt", FMTS)
def test_every_code_is_a_fixed_point(fmt):
    bits = PARAMS[fmt][0]
    for c in range(1 << bits):
        v = O.decode_element(c, fmt)
        if not np.isfinite(v):
            continue
        if fmt == O.INT8 and c == 0x80:
            continue  # -2 is never produced: symmetric saturation
        for mode in (O.RNE, O.RHAZ):
            got = O.encode_element(v, fmt, mode)
            if fmt != O.INT8 or c != 0:
                assert got == c, (fmt, c, got)


@pytest.mark.parametrize("fmt", FP_FMTS)
def test_rne_matches_ml_dtypes_cast(fmt):
    rng = np.random.default_rng(fmt + 11)
    mx = PARAMS[fmt][2]
    x = np.concatenate([
        rng.uniform(-mx, mx, 20000),
        rng.standard_normal(20000) * mx / 50,
        rng.standard_normal(5000) * 2.0 ** -8,
    ]).astype(np.float32)
    x = np.clip(x, -mx, mx)  # ml_dtypes does not saturate
    lib_codes = x.astype(ML[fmt]).view(np.uint8)
    mine = np.array([O.encode_element(float(v), fmt, O.RNE) for v in x], dtype=np.uint8)
    mask = (1 << PARAMS[fmt][0]) - 1
    assert ((lib_codes & mask) == mine).all()


@pytest.mark.parametrize("fmt", FMTS)
def test_saturation_and_forbidden_codes(fmt):
    bits, emax, mx = PARAMS[fmt]
    top_code = O.encode_element(mx, fmt, O.RNE)
    for r in np.linspace(mx, 2.0 ** (emax + 1), 257)[:-1]:
        for mode in (O.RNE, O.RHAZ):
            assert O.encode_element(float(r), fmt, mode) == top_code
            neg = O.encode_element(-float(r), fmt, mode)
            assert O.decode_element(neg, fmt) == -mx
    assert O.decode_element(top_code, fmt) == mx
    forbidden = {O.E4M3: {0x7F, 0xFF}, O.E5M2: set(range(0x7C, 0x80)) | set(range(0xFC, 0x100)),
                 O.INT8: {0x80}}.get(fmt, set())
    rng = np.random.default_rng(5)
    x = (rng.standard_normal((64, 256)) * np.exp(rng.standard_normal((64, 256)) * 3)).astype(np.float32)
    e, _ = O.quantize(x, 1, fmt, O.RHAZ, O.LINEAR)
    codes = O.unpack_codes(e, x.size, fmt)
    assert not (set(np.unique(codes).tolist()) & forbidden)


@pytest.mark.parametrize("fmt", FMTS)
def test_scale_byte_closed_form_and_equivariance(fmt):
    emax = PARAMS[fmt][1]
    rng = np.random.default_rng(3)
    for _ in range(200):
        v = rng.standard_normal(32).astype(np.float32) * np.float32(2.0 ** rng.integers(-60, 60))
        amax = np.abs(v).max()
        codes, sb = O.quantize_block(v, fmt)
        want = int(np.floor(np.log2(float(amax)))) - emax + 127
        assert sb == min(max(want, 0), 254)
        # library special case: E8M0 conversion (round toward zero) of amax is floor(log2) + 127
        assert sb + emax == int(np.array([amax]).astype(ml_dtypes.float8_e8m0fnu).view(np.uint8)[0]) \
            or float(np.array([amax]).astype(ml_dtypes.float8_e8m0fnu).astype(np.float32)[0]) != 2.0 ** np.floor(np.log2(float(amax)))
        j = int(rng.integers(-20, 20))
        codes2, sb2 = O.quantize_block(v * np.float32(2.0 ** j), fmt)
        assert sb2 == sb + j and (codes2 == codes).all()
    # exact powers of two map the block maximum onto 2^emax_elem
    for p in (-100, -3, 0, 5, 100):
        v = np.zeros(32, np.float32)
        v[4] = 2.0 ** p
        codes, sb = O.quantize_block(v, fmt)
        assert sb == p - emax + 127
        assert O.decode_element(int(codes[4]), fmt) == min(2.0 ** emax, PARAMS[fmt][2]) or fmt == O.INT8
        if fmt == O.INT8:
            assert codes[4] == 0x40


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("mode", [O.RNE, O.RHAZ])
def test_error_bound_sign_symmetry_monotone_fixed_point(fmt, mode):
    bits, emax, mx = PARAMS[fmt]
    rng = np.random.default_rng(17 + fmt)
    x = (rng.standard_normal((32, 128)) * np.exp(rng.standard_normal((32, 128)))).astype(np.float32)
    e, s = O.quantize(x, 1, fmt, mode, O.LINEAR)
    d = O.dequantize(e, s, 32, 128, fmt, O.F64, O.LINEAR)
    X = np.repeat(2.0 ** (s.astype(np.float64) - 127), 32).reshape(32, 128)
    r = x.astype(np.float64) / X
    # unsaturated elements are within half a grid step; saturated ones clamp to max normal
    sat = np.abs(r) > mx
    assert (np.abs(d[sat]) == (mx * X)[sat]).all()
    if fmt == O.INT8:
        step = np.full_like(r, 1 / 64)
    else:
        mbits = {O.E4M3: 3, O.E5M2: 2, O.E3M2: 2, O.E2M3: 3, O.E2M1: 1}[fmt]
        emin = {O.E4M3: -6, O.E5M2: -14, O.E3M2: -2, O.E2M3: 0, O.E2M1: 0}[fmt]
        ex = np.floor(np.log2(np.maximum(np.abs(r), 2.0 ** -300)))
        step = 2.0 ** (np.maximum(ex, emin) - mbits)
    assert (np.abs(d - x)[~sat] <= (X * step / 2)[~sat]).all()
    # the block maximum always lands in the top binade: |d| max >= 2^emax * X
    assert (np.abs(d).reshape(32, 4, 32).max(-1) >= (2.0 ** min(emax, np.log2(mx))) * 2.0 ** (s.reshape(32, 4).astype(np.float64) - 127) * (1 - 1e-12)).all()
    # sign symmetry
    e2, s2 = O.quantize(-x, 1, fmt, mode, O.LINEAR)
    d2 = O.dequantize(e2, s2, 32, 128, fmt, O.F64, O.LINEAR)
    assert (s2 == s).all() and (d2 == -d).all()
    # monotone within a block
    order = np.argsort(x.reshape(-1, 32), axis=1)
    dsorted = np.take_along_axis(d.reshape(-1, 32), order, axis=1)
    assert (np.diff(dsorted, axis=1) >= 0).all()
    # re-quantization is a fixed point, bit for bit
    e3, s3 = O.quantize(d.astype(np.float32), 1, fmt, mode, O.LINEAR)
    assert (s3 == s).all() and (e3 == e).all()


def test_zero_flush_clamp_and_nonfinite_blocks():
    for fmt in FMTS:
        z = np.zeros(32, np.float32)
        codes, sb = O.quantize_block(z, fmt)
        assert sb == 0 and not codes.any()
        z[3] = -0.0
        codes, sb = O.quantize_block(z, fmt)
        signcode = 0 if fmt == O.INT8 else 1 << (PARAMS[fmt][0] - 1)
        assert sb == 0 and codes[3] == signcode
        # FP32 subnormals are zeros: block of subnormals is a zero block
        sub = np.full(32, 1e-40, np.float32)
        codes, sb = O.quantize_block(sub, fmt)
        assert sb == 0 and not codes.any()
        # a subnormal next to a normal maximum encodes as zero even when the clamped scale would resolve it
        v = np.zeros(32, np.float32)
        v[0] = 2.0 ** -126
        v[1] = 2.0 ** -127
        codes, sb = O.quantize_block(v, fmt)
        assert sb == max(1 - PARAMS[fmt][1], 0) and codes[1] == 0 and codes[0] != 0
        for bad in (np.inf, -np.inf, np.nan):
            v = np.ones(32, np.float32)
            v[7] = bad
            codes, sb = O.quantize_block(v, fmt)
            assert sb == 0xFF and not codes.any()
            e, s = O.quantize(v.reshape(1, 32), 1, fmt, O.RNE, O.LINEAR)
            d = O.dequantize(e, s, 1, 32, fmt, O.F32, O.LINEAR)
            assert np.isnan(d).all()
            assert (d.view(np.uint32) == 0x7FC00000).all()
            db = O.dequantize(e, s, 1, 32, fmt, O.BF16, O.LINEAR)
            assert (db == 0x7FC0).all()


def test_swizzled_scale_offsets():
    S = O.SWIZZLED
    assert O.scale_offset(0, 0, 256, 8, S) == 0
    assert O.scale_offset(1, 0, 256, 8, S) == 16
    assert O.scale_offset(32, 0, 256, 8, S) == 4
    assert O.scale_offset(0, 1, 256, 8, S) == 1
    assert O.scale_offset(0, 4, 256, 8, S) == 512
    assert O.scale_offset(128, 0, 256, 8, S) == 512 * 2
    assert O.scale_offset(128, 0, 256, 9, S) == 512 * 3
    for rows, kb in ((128, 4), (200, 7), (1, 1), (257, 9)):
        offs = {O.scale_offset(r, k, rows, kb, S) for r in range(rows) for k in range(kb)}
        assert len(offs) == rows * kb
        assert max(offs) < O.scales_bytes(rows, kb, S)
        assert O.scales_bytes(rows, kb, S) == -(-rows // 128) * -(-kb // 4) * 512
    # padding bytes are written as zero
    x = np.ones((3, 64), np.float32)
    _, s = O.quantize(x, 1, O.E4M3, O.RNE, S)
    assert s.size == 512 and np.count_nonzero(s) == 6


def test_axis_semantics_match_quantizing_the_transpose():
    rng = np.random.default_rng(9)
    x = rng.standard_normal((64, 96)).astype(np.float32)
    for fmt in FMTS:
        e0, s0 = O.quantize(x, 0, fmt, O.RNE, O.LINEAR)
        e1, s1 = O.quantize(np.ascontiguousarray(x.T), 1, fmt, O.RNE, O.LINEAR)
        assert (e0 == e1).all() and (s0 == s1).all()
    y = rng.standard_normal((2, 64, 5)).astype(np.float32)
    e0, s0 = O.quantize(y, 1, O.E5M2, O.RHAZ, O.LINEAR)
    yt = np.ascontiguousarray(y.transpose(0, 2, 1)).reshape(10, 64)
    e1, s1 = O.quantize(yt, 1, O.E5M2, O.RHAZ, O.LINEAR)
    assert (e0 == e1).all() and (s0 == s1).all()


def test_bf16_input_equals_widened_fp32_input():
    rng = np.random.default_rng(21)
    x32 = rng.standard_normal((8, 64)).astype(np.float32)
    xb = x32.astype(ml_dtypes.bfloat16)
    wide = xb.astype(np.float32)
    for fmt in FMTS:
        eb, sb = O.quantize(xb.view(np.uint16), 1, fmt, O.RNE, O.LINEAR)
        ef, sf = O.quantize(wide, 1, fmt, O.RNE, O.LINEAR)
        assert (eb == ef).all() and (sb == sf).all()


@pytest.mark.parametrize("fmt", FMTS)
def test_dequantize_values_and_bf16_rounding(fmt):
    rng = np.random.default_rng(33)
    bits = PARAMS[fmt][0]
    n = 4 * 64
    codes = rng.integers(0, 1 << bits, n, dtype=np.uint8)
    elems = O.pack_codes(codes, fmt)
    scales = rng.integers(0, 255, n // 32, dtype=np.uint8)
    scales[0] = 0
    scales[1] = 254
    d64 = O.dequantize(elems, scales, 4, 64, fmt, O.F64, O.LINEAR).reshape(-1)
    d32 = O.dequantize(elems, scales, 4, 64, fmt, O.F32, O.LINEAR).reshape(-1)
    d16 = O.dequantize(elems, scales, 4, 64, fmt, O.BF16, O.LINEAR).reshape(-1)
    for i in range(n):
        p = O.decode_element(int(codes[i]), fmt)
        want = p * 2.0 ** (int(scales[i // 32]) - 127)
        if np.isnan(want):
            assert np.isnan(d64[i]) and np.isnan(d32[i])
            continue
        assert d64[i] == want
        with np.errstate(over="ignore"):
            assert d32[i] == np.float32(want)  # exact or +-Inf beyond the FP32 range
        ref16 = np.float32(want).astype(ml_dtypes.bfloat16).view(np.uint16)
        assert d16[i] == ref16


def test_gemm_closed_forms():
    # all elements +-1 with power-of-two scales: C = K * 2^(a+b) exactly
    M = N = 4
    K = 64
    A = np.ones((M, K), np.float32) * 2.0 ** 3
    B = -np.ones((N, K), np.float32) * 2.0 ** -5
    for fa, fb in itertools.product(FP_FMTS, FP_FMTS):
        ea, sa = O.quantize(A, 1, fa)
        eb, sb = O.quantize(B, 1, fb)
        C, S = O.gemm(ea, sa, eb, sb, M, N, K, fa, fb)
        assert (C == -K * 2.0 ** -2).all() and (S == K * 2.0 ** -2).all()
    # general values: equals numpy's float64 product of the dequantized operands
    rng = np.random.default_rng(2)
    A = rng.standard_normal((8, 96)).astype(np.float32)
    B = rng.standard_normal((12, 96)).astype(np.float32)
    ea, sa = O.quantize(A, 1, O.E4M3)
    eb, sb = O.quantize(B, 1, O.E2M1)
    C, S = O.gemm(ea, sa, eb, sb, 8, 12, 96, O.E4M3, O.E2M1)
    da = O.dequantize(ea, sa, 8, 96, O.E4M3, O.F64)
    db = O.dequantize(eb, sb, 12, 96, O.E2M1, O.F64)
    assert np.allclose(C, da @ db.T, rtol=1e-13, atol=0)
    assert np.allclose(S, np.abs(da) @ np.abs(db).T, rtol=1e-13, atol=0)
    # +1 on one scale byte of a row of A doubles that block's contribution
    off = O.scale_offset(3, 1, 8, 3, O.SWIZZLED)
    sa2 = sa.copy()
    sa2[off] += 1
    C2, _ = O.gemm(ea, sa2, eb, sb, 8, 12, 96, O.E4M3, O.E2M1)
    blk = da[3, 32:64] @ db[:, 32:64].T
    assert np.allclose(C2[3] - C[3], blk, rtol=1e-12, atol=1e-300)
    assert (np.delete(C2, 3, axis=0) == np.delete(C, 3, axis=0)).all()
    # sampled variant agrees with the full one
    ms = np.array([0, 3, 7, 7])
    ns = np.array([0, 11, 5, 0])
    c, s = O.gemm_samples(ea, sa, eb, sb, 8, 12, 96, O.E4M3, O.E2M1, ms, ns)
    assert (c == C[ms, ns]).all() and (s == S[ms, ns]).all()
    # a NaN scale poisons the row
    sa3 = sa.copy()
    sa3[O.scale_offset(2, 0, 8, 3, O.SWIZZLED)] = 0xFF
    C3, _ = O.gemm(ea, sa3, eb, sb, 8, 12, 96, O.E4M3, O.E2M1)
    assert np.isnan(C3[2]).all() and not np.isnan(np.delete(C3, 2, axis=0)).any()


# ---- convolution helpers (the definition written out; pinned to brute force and to a library) ----

def test_conv_oracle_against_brute_force_and_library():
    import torch
    rng = np.random.default_rng(5)
    for (N, H, W, C, Cout, kh, kw, st, pd, dl) in [(1, 5, 6, 3, 2, 3, 3, (1, 1), (1, 1), (1, 1)),
                                                   (2, 7, 5, 4, 3, 3, 2, (2, 1), (0, 2), (1, 2)),
                                                   (1, 4, 4, 2, 2, 1, 1, (1, 1), (0, 0), (1, 1)),
                                                   (1, 9, 8, 2, 1, 2, 3, (3, 2), (2, 1), (2, 1))]:
        x = rng.standard_normal((N, H, W, C))
        w = rng.standard_normal((Cout, kh, kw, C))
        y, s = O.conv2d_nhwc(x, w, st, pd, dl)
        Ho, Wo = O.conv_out_hw(H, W, kh, kw, st, pd, dl)
        assert y.shape == (N, Ho, Wo, Cout)
        # brute force, one output at a time, straight from the formula
        for n in range(N):
            for ho in range(Ho):
                for wo in range(Wo):
                    for co in range(Cout):
                        acc = 0.0
                        acc_abs = 0.0
                        for i in range(kh):
                            for j in range(kw):
                                hi, wi = ho * st[0] - pd[0] + i * dl[0], wo * st[1] - pd[1] + j * dl[1]
                                if 0 <= hi < H and 0 <= wi < W:
                                    acc += float(np.dot(x[n, hi, wi], w[co, i, j]))
                                    acc_abs += float(np.dot(np.abs(x[n, hi, wi]), np.abs(w[co, i, j])))
                        assert abs(acc - y[n, ho, wo, co]) < 1e-12
                        assert abs(acc_abs - s[n, ho, wo, co]) < 1e-12
        # the library routine (channels first)
        ref = torch.nn.functional.conv2d(torch.from_numpy(x).permute(0, 3, 1, 2),
                                         torch.from_numpy(w).permute(0, 3, 1, 2), stride=st, padding=pd,
                                         dilation=dl).permute(0, 2, 3, 1).numpy()
        assert np.allclose(ref, y, atol=1e-12)
        # the gather table agrees with the same index arithmetic done by the library on an index image
        src = O.im2col_source_pixels(N, H, W, kh, kw, st, pd, dl)
        idx_img = torch.arange(1, N * H * W + 1, dtype=torch.float64).view(N, 1, H, W)   # 0 = padding
        cols = torch.nn.functional.unfold(idx_img, (kh, kw), dilation=dl, padding=pd, stride=st)  # [N, kh*kw, Ho*Wo]
        want = cols.permute(0, 2, 1).reshape(N * Ho * Wo, kh * kw).numpy().astype(np.int64) - 1
        assert np.array_equal(src, want)


# ---- partial last block (axis length not a multiple of 32) ----

def test_partial_block_is_the_zero_padded_block():
    """Reading: the missing elements of a last, partial block are +0 and the stored row is padded
    with zero codes.  So quantizing a tensor with a tail must equal quantizing the tensor padded
    with +0.0 to whole blocks (an all-explicit computation the other pins already cover), on either
    axis, and dequantizing must return exactly the unpadded part."""
    rng = np.random.default_rng(11)
    for (R, L) in ((3, 1), (5, 31), (4, 33), (7, 40), (2, 100)):
        Lp = (L + 31) // 32 * 32
        x = (rng.standard_normal((R, L)) * np.exp(rng.standard_normal((R, 1)))).astype(np.float32)
        x[0, -1] = -0.0
        xp = np.zeros((R, Lp), np.float32)
        xp[:, :L] = x
        for fmt in range(6):
            for layout in (O.LINEAR, O.SWIZZLED):
                e, s = O.quantize(x, 1, fmt, O.RHAZ, layout)
                ep, sp = O.quantize(xp, 1, fmt, O.RHAZ, layout)
                assert e.size == R * Lp * O.fmt_bits(fmt) // 8
                assert np.array_equal(e, ep) and np.array_equal(s, sp)
                d = O.dequantize(e, s, R, L, fmt, O.F32, layout)
                dp = O.dequantize(ep, sp, R, Lp, fmt, O.F32, layout)
                assert d.shape == (R, L) and np.array_equal(d.view(np.uint32), dp[:, :L].view(np.uint32))
            # blocks along axis 0 of the transposed tensor: the same codes, row for row
            et, st = O.quantize(np.ascontiguousarray(x.T), 0, fmt, O.RNE, O.LINEAR)
            e1, s1 = O.quantize(x, 1, fmt, O.RNE, O.LINEAR)
            assert np.array_equal(et, e1) and np.array_equal(st, s1)


def test_partial_block_worked_example():
    """Eight elements: the scale comes from the largest of the eight, positions 8..31 hold code 0."""
    v = np.array([[1.0, -2.0, 3.0, 0.5, 96.0, -0.25, 7.0, 12.0]], np.float32)
    e, s = O.quantize(v, 1, O.E4M3, O.RNE, O.LINEAR)
    assert s.tolist() == [127 + 6 - 8]                      # floor(log2 96) = 6, emax(E4M3) = 8
    codes = O.unpack_codes(e, 32, O.E4M3)
    assert (codes[8:] == 0).all()
    X = 2.0 ** (6 - 8)
    assert [O.decode_element(int(c), O.E4M3) * X for c in codes[:8]] == v[0].tolist()   # all exactly representable
