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
