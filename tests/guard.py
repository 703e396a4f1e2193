"""Output buffers with a canary behind them (test helper, no test of its own).

Every tensor handed out is followed in device memory by 64 bytes of a fixed pattern; `check()`
asserts that no kernel wrote past the end of any of them.  It stands in for a memory checker on the
outputs and the workspace of the contraction and quantizer calls.
"""
import math

import torch

CANARY_BYTES = 64
PATTERN = 0xC3


class Guard:
    def __init__(self, device="cuda"):
        self.device = device
        self._tails = []

    def alloc(self, shape, dtype, fill=None):
        """A contiguous tensor of `shape` whose last byte is directly followed by the canary."""
        shape = (shape,) if isinstance(shape, int) else tuple(shape)
        item = torch.empty((), dtype=dtype).element_size()
        nbytes = math.prod(shape) * item
        raw = torch.empty(nbytes + CANARY_BYTES, dtype=torch.uint8, device=self.device)
        raw[nbytes:] = PATTERN
        self._tails.append((raw, nbytes))
        t = raw[:nbytes].view(dtype).view(shape)
        if fill is not None:
            t.fill_(fill)
        return t

    def check(self):
        for raw, nbytes in self._tails:
            tail = raw[nbytes:]
            assert bool((tail == PATTERN).all()), "a kernel wrote past the end of a %d-byte buffer" % nbytes
