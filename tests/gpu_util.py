"""Helpers shared by the GPU parity tests: moving the same bytes to both sides
and guard bands around every output buffer."""
import numpy as np
import torch

GUARD = 4096


def to_oracle_input(x: torch.Tensor) -> np.ndarray:
    """The tensor's bytes as the oracle takes them (float32, or uint16 for BF16)."""
    x = x.detach().cpu().contiguous()
    if x.dtype == torch.bfloat16:
        return x.view(torch.int16).numpy().view(np.uint16)
    return x.numpy()


class Guarded:
    """A device buffer with 4 KiB of 0xA5 before and after the part handed out."""

    def __init__(self, nbytes: int, device="cuda"):
        self.n = nbytes
        self.raw = torch.full((nbytes + 2 * GUARD,), 0xA5, dtype=torch.uint8, device=device)
        self.view = self.raw[GUARD:GUARD + nbytes]
        assert self.view.data_ptr() % 256 == 0

    def check(self):
        assert bool((self.raw[:GUARD] == 0xA5).all()), "write before the buffer"
        assert bool((self.raw[GUARD + self.n:] == 0xA5).all()), "write past the buffer"


def sample_rows(n: int, count: int = 256, seed: int = 0) -> np.ndarray:
    """`count` row indices of a tensor with n rows: both ends, the seams of the 32- / 128- / 256-row
    tiles the kernels work in, and random rows from the middle.  Sorted, unique."""
    picks = [0, 1, 2, 3, n - 4, n - 3, n - 2, n - 1]
    for seam in (32, 128, 256, 1024, n // 2, n - 256, n - 128, n - 32):
        picks += [seam - 1, seam, seam + 1]
    rng = np.random.default_rng(seed)
    picks = [p for p in picks if 0 <= p < n]
    rest = rng.choice(n, size=min(n, count), replace=False)
    sel = np.unique(np.concatenate([np.array(picks, dtype=np.int64), rest]))
    if sel.size > count:   # keep every hand-picked row, thin out the random ones
        keep = np.isin(sel, picks)
        extra = sel[~keep][: count - int(keep.sum())]
        sel = np.unique(np.concatenate([sel[keep], extra]))
    return sel


def swizzled_scale_offsets(rows_idx: np.ndarray, rows: int, kblocks: int) -> np.ndarray:
    """Byte offsets [len(rows_idx), kblocks] of the scales of the given rows in the swizzled
    tensor (512-byte chunks of 128 rows x 4 blocks, chunks K-fastest): the layout the header
    defines, written out for whole rows at once."""
    r = np.asarray(rows_idx, dtype=np.int64).reshape(-1, 1)
    k = np.arange(kblocks, dtype=np.int64).reshape(1, -1)
    return ((r // 128) * ((kblocks + 3) // 4) + k // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + k % 4


def assert_operand_rows_match_oracle(O, x: torch.Tensor, axis: int, fmt: int, rounding: int,
                                     elems: torch.Tensor, scales: torch.Tensor, what: str,
                                     count: int = 256, seed: int = 0):
    """Byte comparison of a GPU-quantized 2-D operand (K-major codes, SWIZZLED scales) with the
    oracle on `count` sampled output rows.  Output row j is input row j (axis 1) or input column j
    (axis 0); rows of an MX tensor are independent, so the oracle quantizes just the sampled
    rows / columns of the very same input bytes."""
    assert x.dim() == 2 and axis in (0, 1)
    n_rows = x.shape[1 - axis]
    L = x.shape[axis]
    kblocks = (L + 31) // 32
    sel = sample_rows(n_rows, count, seed)
    sel_t = torch.from_numpy(sel).to(x.device)
    if axis == 1:
        sub = x[sel_t].contiguous()            # [count, L], blocks along the last axis
        want_e, want_s = O.quantize(to_oracle_input(sub), 1, fmt, rounding, O.LINEAR)
    else:
        sub = x[:, sel_t].contiguous()         # [L, count], blocks along axis 0
        want_e, want_s = O.quantize(to_oracle_input(sub), 0, fmt, rounding, O.LINEAR)
    row_bytes = kblocks * 32 * O.fmt_bits(fmt) // 8
    got_e = elems.view(n_rows, row_bytes)[sel_t].cpu().numpy().reshape(-1)
    off = swizzled_scale_offsets(sel, n_rows, kblocks)
    # the offset formula restated above agrees with the oracle's own on a few entries
    for i, kb in ((0, 0), (len(sel) // 2, kblocks // 2), (len(sel) - 1, kblocks - 1)):
        assert off[i, kb] == O.scale_offset(int(sel[i]), kb, n_rows, kblocks, O.SWIZZLED)
    got_s = scales[torch.from_numpy(off.reshape(-1)).to(x.device)].cpu().numpy()
    if not np.array_equal(got_e, want_e):
        bad = np.flatnonzero(got_e != want_e)
        raise AssertionError(f"{what}: {bad.size} code bytes differ from the oracle; first in sampled row "
                             f"{sel[bad[0] // row_bytes]} at byte {bad[0] % row_bytes}")
    if not np.array_equal(got_s, want_s):
        bad = np.flatnonzero(got_s != want_s)
        raise AssertionError(f"{what}: {bad.size} scale bytes differ from the oracle; first in sampled row "
                             f"{sel[bad[0] // kblocks]} block {bad[0] % kblocks}")
