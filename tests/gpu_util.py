"""Helpers for the GPU parity tests: a library session on a torch-allocated heap, and
mirrored buffers that exist both in the CUDA library's symmetric heap and in the CPU
oracle's heap, so that the same seeded inputs can be handed to both sides."""
from __future__ import annotations

import numpy as np
import torch

from oracle import Oracle
from paper_2409_20476_b200 import binding as B


class Session:
    """``npes`` PEs on a heap owned by a torch tensor (PyTorch only supplies the memory)."""

    def __init__(self, npes: int, heap_bytes: int, with_oracle: bool = True):
        assert torch.cuda.is_available()
        heap_bytes = (heap_bytes + 255) // 256 * 256
        self.npes, self.heap_bytes = npes, heap_bytes
        self.heap = torch.zeros(npes * heap_bytes, dtype=torch.uint8, device="cuda")
        torch.cuda.synchronize()
        B.ishmemx_init_external(npes, heap_bytes, self.heap.data_ptr())
        self.base = self.heap.data_ptr()
        self.oracle = Oracle(npes, heap_bytes) if with_oracle else None
        self.open = True
        self.same_layout = True

    def close(self):
        if self.open:
            B.ishmem_finalize()
            self.open = False
            if self.oracle is not None:
                self.oracle.close()
            del self.heap
            torch.cuda.empty_cache()

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # -- symmetric buffers mirrored on both sides ------------------------------------------
    def malloc(self, nbytes: int) -> "Sym":
        addr = B.ishmem_malloc(nbytes)
        assert addr, "symmetric heap exhausted"
        ooff = self.oracle.malloc(nbytes) if self.oracle is not None else None
        if ooff is not None and ooff != addr - self.base:
            self.same_layout = False
        return Sym(self, addr, nbytes, ooff)

    def sync(self):
        torch.cuda.synchronize()

    def status(self, clear=True) -> int:
        return B.ishmemx_status(1 if clear else 0)


class Sym:
    """One symmetric object: GPU address (PE 0's copy), oracle offset, size."""

    def __init__(self, s: Session, addr: int, nbytes: int, ooff):
        self.s, self.addr, self.nbytes, self.ooff = s, addr, nbytes, ooff
        self.off = addr - s.base

    def gpu(self, pe: int, dtype=torch.uint8) -> torch.Tensor:
        lo = pe * self.s.heap_bytes + self.off
        return self.s.heap[lo:lo + self.nbytes].view(dtype)

    def cpu(self, pe: int, dtype=np.uint8) -> np.ndarray:
        return self.s.oracle.view(self.ooff, self.nbytes, pe, dtype)

    def fill(self, pe: int, data: np.ndarray):
        """Write the same bytes into the GPU heap and the oracle heap."""
        raw = np.ascontiguousarray(data).view(np.uint8).ravel()
        assert raw.size <= self.nbytes
        self.gpu(pe)[:raw.size].copy_(torch.from_numpy(raw.copy()))
        if self.s.oracle is not None:
            self.cpu(pe)[:raw.size] = raw

    def read(self, pe: int, dtype=np.uint8) -> np.ndarray:
        torch.cuda.synchronize()
        return self.gpu(pe).cpu().numpy().view(dtype)

    def assert_equal(self, what=""):
        """Bit-exact comparison of every PE's copy with the oracle's."""
        torch.cuda.synchronize()
        for pe in range(self.s.npes):
            got = self.gpu(pe).cpu().numpy()
            exp = self.cpu(pe)
            if not np.array_equal(got, exp):
                bad = np.nonzero(got != exp)[0]
                raise AssertionError(f"{what}: PE {pe} differs at {bad.size} bytes, first at {bad[0]}"
                                     f" (got {got[bad[0]]}, oracle {exp[bad[0]]})")


def heaps_equal(s: Session, what=""):
    """Whole-heap comparison (small heaps only): nothing outside the targets was touched."""
    torch.cuda.synchronize()
    assert s.same_layout, "whole-heap comparison needs identical offsets on both sides"
    for pe in range(s.npes):
        got = s.heap[pe * s.heap_bytes:(pe + 1) * s.heap_bytes].cpu().numpy()
        exp = s.oracle.view(0, s.heap_bytes, pe)
        if not np.array_equal(got, exp):
            bad = np.nonzero(got != exp)[0]
            raise AssertionError(f"{what}: PE {pe} heap differs at {bad.size} bytes, first at offset {bad[0]}")
