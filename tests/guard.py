"""Guard bands around device buffers (the stand-in for a memory checker on a box where none can run).

Every buffer handed out here sits in the middle of a larger allocation whose margins are filled with a
canary byte; `check()` verifies that the margins still hold it.  A kernel that writes a few rows past the
end of an output, or scribbles before or behind its workspace, fails the test that ran it instead of
corrupting a neighbour silently.  (Reads out of bounds are not caught; wild writes further than a band
away are not either.)
"""
import torch

BAND = 64 << 10   # bytes on each side
CANARY = 0xC3


class Guards:
    def __init__(self, device="cuda"):
        self.device = device
        self.raw = []

    def _carve(self, nbytes: int) -> torch.Tensor:
        nbytes = max(int(nbytes), 256)
        raw = torch.full((nbytes + 2 * BAND,), CANARY, dtype=torch.uint8, device=self.device)
        self.raw.append((raw, nbytes))
        return raw[BAND:BAND + nbytes]          # BAND is a multiple of 256: alignment is kept

    def workspace(self, nbytes: int, device=None) -> torch.Tensor:
        return self._carve(nbytes)

    def empty(self, shape, dtype) -> torch.Tensor:
        n = 1
        for s in shape:
            n *= int(s)
        es = torch.empty((), dtype=dtype).element_size()
        return self._carve(n * es)[:n * es].view(dtype).view(*shape)

    def empty_like(self, t: torch.Tensor) -> torch.Tensor:
        return self.empty(tuple(t.shape), t.dtype)

    def check(self) -> None:
        torch.cuda.synchronize()
        for raw, nbytes in self.raw:
            lo, hi = raw[:BAND], raw[BAND + nbytes:]
            assert bool((lo == CANARY).all()), f"bytes before a {nbytes}-byte buffer were overwritten"
            assert bool((hi == CANARY).all()), f"bytes behind a {nbytes}-byte buffer were overwritten"
        self.raw.clear()
