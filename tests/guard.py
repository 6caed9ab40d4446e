"""Poisoned, fenced device buffers for the GPU tests (a stand-in for a memory checker).

Every output or scratch tensor handed to the library is carved out of a larger allocation that is
filled with the byte 0xFF: the tensor's own bytes read as NaN in bf16 and fp32 (and as -1 in int32),
and a guard band of the same pattern lies before and after it.  After a call the test asserts that

  * the guard bands are byte for byte untouched (nothing was written outside the tensor), and
  * no element of an output still holds the pattern (nothing was left unwritten).

Inputs can be fenced the same way: a read that strays into a band brings NaNs into the result,
which the finiteness check of the comparison then sees.
"""
import torch

POISON = 0xFF
ALIGN = 256


class Fenced:
    """One tensor of `shape`/`dtype` with `guard_bytes` of poison on either side."""

    def __init__(self, shape, dtype, guard_bytes=1 << 20, device="cuda", fill_from=None):
        numel = 1
        for s in shape:
            numel *= int(s)
        self.nbytes = numel * torch.empty((), dtype=dtype).element_size()
        guard = (int(guard_bytes) + ALIGN - 1) // ALIGN * ALIGN
        total = guard + (self.nbytes + ALIGN - 1) // ALIGN * ALIGN + guard + ALIGN
        self.raw = torch.full((total,), POISON, dtype=torch.uint8, device=device)
        base = self.raw.data_ptr()
        self.start = (-base) % ALIGN + guard                      # the interior starts on a 256-byte boundary
        self.t = self.raw[self.start:self.start + self.nbytes].view(dtype).view(*shape)
        assert self.t.data_ptr() % ALIGN == 0
        if fill_from is not None:
            self.t.copy_(fill_from)

    def guards_intact(self) -> bool:
        before = self.raw[:self.start]
        after = self.raw[self.start + self.nbytes:]
        return bool((before == POISON).all().item()) and bool((after == POISON).all().item())

    def fully_written(self) -> bool:
        """No element still holds the poison pattern (NaN for floating types, -1 for integers)."""
        if self.t.dtype.is_floating_point:
            return not bool(torch.isnan(self.t).any().item())
        return not bool((self.t.view(torch.uint8) == POISON).view(-1, self.t.element_size()).all(dim=1).any().item())

    def untouched(self) -> bool:
        """Every byte of the tensor itself still holds the pattern."""
        return bool((self.raw[self.start:self.start + self.nbytes] == POISON).all().item())

    def check(self, name, written=True):
        assert self.guards_intact(), f"{name}: bytes outside the tensor were written"
        if written:
            assert self.fully_written(), f"{name}: some elements were never written"
