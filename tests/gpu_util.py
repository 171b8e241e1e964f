"""Helpers of the GPU parity tests: device buffers with guard words around every output,
and bit-pattern comparisons against the CPU checker's results."""
import numpy as np
import torch

GUARD_WORDS = 64          # 256 bytes on each side, keeps the payload 16-byte aligned
GUARD_PATTERN = 0x5A5A5A5A


class Guarded:
    """A device buffer of `n` 32-bit words with guard words before and after it."""

    def __init__(self, n, dtype, fill=None):
        assert dtype in (torch.float32, torch.int32)
        self.n = n
        self.raw = torch.full((n + 2 * GUARD_WORDS,), GUARD_PATTERN, dtype=torch.int32, device="cuda")
        self.view = self.raw[GUARD_WORDS:GUARD_WORDS + n].view(dtype)
        if fill is not None:
            self.view.copy_(torch.from_numpy(np.ascontiguousarray(fill)).view(dtype))
        else:
            self.view.view(torch.int32).fill_(0x7FC0DEAD)   # poison: unwritten outputs show up

    def check_guards(self):
        r = self.raw.cpu().numpy()
        assert (r[:GUARD_WORDS] == GUARD_PATTERN).all(), "write before the buffer"
        assert (r[GUARD_WORDS + self.n:] == GUARD_PATTERN).all(), "write past the buffer"

    def numpy(self, dtype):
        return self.view.cpu().numpy().view(dtype)


def to_dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def bits_equal(a, b):
    """Number of elements whose 32-bit patterns differ."""
    return int((np.ascontiguousarray(a).view(np.uint32) != np.ascontiguousarray(b).view(np.uint32)).sum())


def max_rel_err(a, b):
    a = a.astype(np.float64)
    b = b.astype(np.float64)
    den = np.maximum(np.abs(a), np.abs(b))
    den[den == 0] = 1.0
    return float((np.abs(a - b) / den).max()) if a.size else 0.0
