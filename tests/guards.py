"""Guard bands around device buffers (a stand-in for a memory checker): every tensor handed to the library
sits in the middle of a larger allocation whose first and last 256 bytes hold a pattern; a kernel that
writes before or behind a buffer it was given shows up as a damaged pattern."""
import math

import torch

GUARD_BYTES = 256
PATTERN = 0xA5


class Guarded:
    def __init__(self, shape, dtype, device, fill=None):
        n = math.prod(shape) * torch.empty((), dtype=dtype).element_size()
        self.raw = torch.full((n + 2 * GUARD_BYTES,), PATTERN, dtype=torch.uint8, device=device)
        self.t = self.raw[GUARD_BYTES:GUARD_BYTES + n].view(dtype).view(*shape)
        if fill is None:
            self.t.zero_()
        else:
            self.t.copy_(fill)

    def intact(self) -> bool:
        lo = self.raw[:GUARD_BYTES]
        hi = self.raw[-GUARD_BYTES:]
        return bool((lo == PATTERN).all().item()) and bool((hi == PATTERN).all().item())


def all_intact(items) -> bool:
    return all(g.intact() for g in items)
