"""Helpers of the GPU tests: guarded device buffers and the tests-only builds of the library.

Guarded buffers stand in for a memory checker on the write side: every device buffer a test hands to the
library sits between two guard bands of GUARD bytes filled with a pattern; after the call the bands must be
untouched, so a kernel that writes before or past a buffer fails the test that ran it.  (The read side is
covered by the checking build, see checked_library.)
"""
import contextlib

import numpy as np

GUARD = 512           # bytes either side; a multiple of 256 keeps the alignment torch gives the allocation
PATTERN = 0xC7


class Guarded:
    """A device buffer of `nbytes` bytes between two guard bands."""

    def __init__(self, torch, nbytes: int, fill=None):
        self.torch = torch
        self.nbytes = int(nbytes)
        self.raw = torch.full((self.nbytes + 2 * GUARD,), PATTERN, dtype=torch.uint8, device="cuda")
        self.bytes = self.raw[GUARD:GUARD + self.nbytes]
        if fill is not None:
            self.bytes.fill_(fill)

    def view(self, dtype):
        return self.bytes.view(dtype)

    def check(self, what: str = "buffer") -> None:
        head = self.raw[:GUARD]
        tail = self.raw[GUARD + self.nbytes:]
        assert bool((head == PATTERN).all()), f"{what}: bytes before the buffer were overwritten"
        assert bool((tail == PATTERN).all()), f"{what}: bytes past the buffer were overwritten"


def guarded_stream(A, torch, p, fill=0xA5):
    """Stream buffer of exactly the compressed size, stale bytes inside, guards outside."""
    size = A.accept_mbq_compressed_size(p) if isinstance(p, A.MbqParams) else A.accept_compressed_size(p)
    return Guarded(torch, size, fill)


def guarded_workspace(A, torch, p, nbytes=None):
    size = nbytes if nbytes is not None else (
        A.accept_mbq_workspace_size(p) if isinstance(p, A.MbqParams) else A.accept_workspace_size(p))
    return Guarded(torch, size, 0)


def guarded_floats(torch, n: int, value=float("nan")):
    g = Guarded(torch, 4 * n)
    g.view(torch.float32).fill_(value)
    return g


def guarded_input(torch, x_np):
    g = Guarded(torch, 4 * x_np.size)
    g.view(torch.float32).copy_(torch.from_numpy(np.ascontiguousarray(x_np, dtype=np.float32).reshape(-1)))
    return g


@contextlib.contextmanager
def library_variant(name: str):
    """Routes the binding to a tests-only build of the library ("bounds" or "stall") for the duration."""
    from paper_2311_05827_b200 import binding, build
    variant = binding.load(build.build_variant(name))
    binding.lib()  # make sure the product is loaded first, so that it is what comes back
    saved = binding._lib
    binding._lib = variant
    try:
        yield variant
    finally:
        binding._lib = saved
