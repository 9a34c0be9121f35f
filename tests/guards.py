"""Guard regions for the GPU tests: a tensor that a kernel writes or reads is carved out of a larger buffer whose
bytes either side hold a pattern, and the pattern is checked after the kernel has run.  A store or a copy that
lands outside the tensor shows up here even when it does not fault and nothing else reads those bytes."""
import math

import torch

CANARY = 0xA5
PAD_BYTES = 8192          # either side; a multiple of 256, so that the carved tensor keeps its alignment


class Guarded:
    def __init__(self, shape, dtype, device, like: torch.Tensor = None):
        self.nbytes = math.prod(shape) * torch.empty((), dtype=dtype).element_size()
        body = (self.nbytes + 255) // 256 * 256
        self.buf = torch.full((2 * PAD_BYTES + body,), CANARY, dtype=torch.uint8, device=device)
        self.t = self.buf[PAD_BYTES : PAD_BYTES + self.nbytes].view(dtype).view(shape)
        if like is not None:
            self.t.copy_(like)

    def check(self, what: str = ""):
        """Call after the device has finished: every guard byte still holds the pattern."""
        head = self.buf[:PAD_BYTES]
        tail = self.buf[PAD_BYTES + self.nbytes :]
        assert bool((head == CANARY).all()), f"{what}: bytes in front of the tensor were written"
        assert bool((tail == CANARY).all()), f"{what}: bytes behind the tensor were written"
