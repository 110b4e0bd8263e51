"""Guard bands for the GPU tests: every output and workspace handed to the library can be carved out of a larger
allocation whose margins hold a sentinel pattern; after the call the margins must be untouched.  This is the
out-of-bounds-write detector of the test-suite (a memory checker cannot be run on the GPUs these tests use)."""
import torch

GUARD_BYTES = 4096
SENTINEL = 0xA5


class Guarded:
    def __init__(self):
        self._bufs = []

    def empty(self, shape, dtype, fill=None, device="cuda"):
        """A tensor of `shape` with GUARD_BYTES of sentinel before and after it (256-byte aligned start)."""
        n = int(torch.Size(shape).numel()) * torch.empty((), dtype=dtype).element_size()
        inner = (n + 255) // 256 * 256
        raw = torch.full((GUARD_BYTES + inner + GUARD_BYTES,), SENTINEL, dtype=torch.uint8, device=device)
        view = raw[GUARD_BYTES:GUARD_BYTES + n].view(dtype).view(shape)
        if fill is not None:
            view.fill_(fill)
        self._bufs.append((raw, n))
        return view

    def check(self):
        torch.cuda.synchronize()
        for i, (raw, n) in enumerate(self._bufs):
            assert bool((raw[:GUARD_BYTES] == SENTINEL).all()), f"buffer {i}: bytes before the tensor were written"
            assert bool((raw[GUARD_BYTES + n:] == SENTINEL).all()), f"buffer {i}: bytes after the tensor were written"
