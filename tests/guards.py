"""Device buffers with a filled guard region before and after the payload (host-side helper of the GPU tests).

A kernel that stores past either end of an output or of the workspace changes guard bytes, which `check()` finds;
this stands in for an out-of-bounds checker.  The payload starts as all-ones bytes (NaN in both floating-point
formats), so an output element left unwritten, or a workspace word read before it is written, shows up as NaN in the
compared result.  No method arithmetic here."""
from __future__ import annotations

import torch

GUARD_BYTES = 4096          # a multiple of every alignment the library asks for
FILL = 0xA5
PAYLOAD = 0xFF              # all-ones bytes are NaN as fp32 and as bf16: a payload element read before it is written shows


class Guarded:
    def __init__(self, shape, dtype, device="cuda"):
        shape = tuple(int(s) for s in shape)
        n = 1
        for s in shape:
            n *= s
        self.nbytes = n * torch.empty((), dtype=dtype).element_size()
        self.buf = torch.full((2 * GUARD_BYTES + self.nbytes,), FILL, dtype=torch.uint8, device=device)
        self.buf[GUARD_BYTES:GUARD_BYTES + self.nbytes] = PAYLOAD
        self.t = self.buf[GUARD_BYTES:GUARD_BYTES + self.nbytes].view(dtype).view(shape)

    def check(self, what=""):
        head, tail = self.buf[:GUARD_BYTES], self.buf[GUARD_BYTES + self.nbytes:]
        assert bool((head == FILL).all()), f"{what}: bytes before the buffer were overwritten"
        assert bool((tail == FILL).all()), f"{what}: bytes after the buffer were overwritten"
