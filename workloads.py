"""Seeded synthetic inputs shaped like the paper's transformer workloads.

The paper (arXiv 2310.10537, Sections 4.3-4.5) measures on trained language
models whose weights and data are not available; these generators stand in for
them with the tensor shapes, value distributions and block structure of the five
benchmark configurations.  The module holds no MX arithmetic: it only draws
random numbers and places zero / tiny blocks.  Both the CUDA tests and the CPU
oracle tests take their inputs from here (generate once, copy the bytes to the
other side).
"""
from __future__ import annotations

import torch

BLOCK = 32


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def student_t(shape, df: int, gen: torch.Generator, device) -> torch.Tensor:
    """Student-t(df) = Z0 / sqrt((Z1^2 + ... + Z_df^2) / df), FP32."""
    z0 = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    chi = torch.zeros(shape, device=device, dtype=torch.float32)
    for _ in range(df):
        z = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
        chi.addcmul_(z, z)
    return z0 / torch.sqrt(chi / df)


def config1(device="cpu", m: int = 256, n: int = 256, k: int = 1024, seed: int = 1001):
    """A FP32 [m x k], B FP32 [k x n], N(0,1); 1% of entries x100; one all-zero
    block per row of A (block (7*i) mod (k/32) of row i)."""
    g = _gen(seed, device)
    out = {}
    for name, shape in (("A", (m, k)), ("B", (k, n))):
        x = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
        mask = torch.rand(shape, generator=g, device=device) < 0.01
        x = torch.where(mask, x * 100.0, x)
        out[name] = x
    a = out["A"].view(m, k // BLOCK, BLOCK)
    rows = torch.arange(m, device=device)
    a[rows, (7 * rows) % (k // BLOCK)] = 0.0
    return out


def config2(device="cpu", rows: int = 8192, cols: int = 8192, seed: int = 2002) -> torch.Tensor:
    """BF16 [rows x cols] = 4 * Student-t(3); 0.1% of the 32-blocks zeroed and a
    disjoint 0.1% scaled down to about 1e-30 in magnitude."""
    g = _gen(seed, device)
    x = 4.0 * student_t((rows, cols), 3, g, device)
    xb = x.view(rows, cols // BLOCK, BLOCK)
    u = torch.rand((rows, cols // BLOCK), generator=g, device=device)
    zero = u < 0.001
    tiny = (u >= 0.001) & (u < 0.002)
    xb[tiny] = xb[tiny] * 2.5e-31
    xb[zero] = 0.0
    return x.to(torch.bfloat16)


def config3(device="cpu", tokens: int = 8192, d_in: int = 4096, d_out: int = 16384,
            seed: int = 3003):
    """FFN up-projection: X BF16 [tokens x d_in] ~ N(0,1), W BF16 [d_in x d_out] ~ N(0, 0.02^2)."""
    g = _gen(seed, device)
    x = torch.randn((tokens, d_in), generator=g, device=device, dtype=torch.float32)
    w = torch.randn((d_in, d_out), generator=g, device=device, dtype=torch.float32) * 0.02
    return {"X": x.to(torch.bfloat16), "W": w.to(torch.bfloat16)}


def config4(device="cpu", n: int = 4096, dtype=torch.float32, seed: int = 4004):
    """One linear layer's training step: X ~ N(0,1), W ~ N(0, 0.02^2), dY ~ N(0, 1e-3^2), all [n x n]."""
    g = _gen(seed, device)
    x = torch.randn((n, n), generator=g, device=device, dtype=torch.float32)
    w = torch.randn((n, n), generator=g, device=device, dtype=torch.float32) * 0.02
    dy = torch.randn((n, n), generator=g, device=device, dtype=torch.float32) * 1e-3
    return {"X": x.to(dtype), "W": w.to(dtype), "dY": dy.to(dtype)}


def config5(device="cpu", tokens: int = 16384, d_in: int = 8192, d_out: int = 28672,
            seed: int = 5005):
    """FP4-weight x FP8-activation: W BF16 [d_in x d_out] ~ N(0, 0.02^2), X BF16 [tokens x d_in] ~ Student-t(5)."""
    g = _gen(seed, device)
    w = torch.randn((d_in, d_out), generator=g, device=device, dtype=torch.float32) * 0.02
    x = student_t((tokens, d_in), 5, g, device)
    return {"W": w.to(torch.bfloat16), "X": x.to(torch.bfloat16)}


def adversarial(device="cpu", rows: int = 96, cols: int = 256, dtype=torch.float32,
                seed: int = 7, nonfinite: bool = True) -> torch.Tensor:
    """A small tensor whose blocks cover the degenerate cases of the conversion:
    zero blocks, negative zeros, FP32/BF16 subnormals, magnitudes near the ends
    of the exponent range, exact powers of two, ties, and (optionally) Inf / NaN."""
    g = _gen(seed, device)
    x = torch.randn((rows, cols), generator=g, device=device, dtype=torch.float32)
    nb = cols // BLOCK
    xb = x.view(rows, nb, BLOCK)
    # per-block magnitude: exponents spread over the whole FP32 range
    e = torch.randint(-126, 127, (rows, nb), generator=g, device=device).to(torch.float32)
    xb.mul_(torch.pow(torch.tensor(2.0, device=device), e).unsqueeze(-1))
    kind = torch.randint(0, 16, (rows, nb), generator=g, device=device)
    xb[kind == 0] = 0.0
    xb[kind == 1] = -0.0
    # exact powers of two and half-way values inside a block
    pw = torch.pow(torch.tensor(2.0, device=device),
                   torch.randint(-8, 8, (rows, nb, BLOCK), generator=g, device=device).to(torch.float32))
    sel = (kind == 2).unsqueeze(-1).expand_as(xb)
    xb[sel] = pw[sel]
    q = torch.randint(-64, 65, (rows, nb, BLOCK), generator=g, device=device).to(torch.float32) / 16.0
    sel = (kind == 3).unsqueeze(-1).expand_as(xb)
    xb[sel] = q[sel]
    # subnormal inputs
    sub = torch.randint(-(1 << 22), 1 << 22, (rows, nb, BLOCK), generator=g, device=device).to(torch.float32) * 2.0 ** -149
    sel = (kind == 4).unsqueeze(-1).expand_as(xb)
    xb[sel] = sub[sel]
    # a block whose maximum is the smallest normal, with subnormal neighbours
    sel5 = kind == 5
    xb[sel5] = xb[sel5].sign() * 2.0 ** -140
    idx = sel5.nonzero()
    if idx.numel():
        xb[idx[:, 0], idx[:, 1], 3] = 2.0 ** -126
        xb[idx[:, 0], idx[:, 1], 9] = -1.75 * 2.0 ** -126
    # near the top of the range
    sel6 = kind == 6
    xb[sel6] = xb[sel6].sign() * torch.finfo(torch.float32).max * 0.75
    if nonfinite:
        idx = (kind == 7).nonzero()
        if idx.numel():
            xb[idx[:, 0], idx[:, 1], 5] = float("inf")
        idx = (kind == 8).nonzero()
        if idx.numel():
            xb[idx[:, 0], idx[:, 1], 17] = float("nan")
        idx = (kind == 9).nonzero()
        if idx.numel():
            xb[idx[:, 0], idx[:, 1], 31] = float("-inf")
    return x.to(dtype)
