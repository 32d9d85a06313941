"""ctypes front end of the sequential CPU oracle (``ishmem_oracle.c``).

Test infrastructure only: tests, the smoke check and the benchmark's CPU legs
may import this; the CUDA library never does, and this module never imports the
CUDA package.  Symmetric objects are named by their byte offset in the heap.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "ishmem_oracle.c"
_LIB = _HERE / "libishmem_oracle.so"

# element types / operators / comparisons: the oracle's own numbering
(T_INT32, T_INT64, T_FLOAT, T_DOUBLE, T_UINT32, T_UINT64, T_INT8, T_UINT8, T_INT16,
 T_UINT16) = range(10)
R_SUM, R_MAX, R_MIN, R_PROD, R_AND, R_OR, R_XOR = range(7)
(A_FETCH_ADD, A_ADD, A_FETCH_INC, A_INC, A_FETCH, A_SET, A_SWAP, A_COMPARE_SWAP,
 A_FETCH_AND, A_FETCH_OR, A_FETCH_XOR) = range(11)
SIG_SET, SIG_ADD = 0, 1
C_EQ, C_NE, C_GT, C_GE, C_LT, C_LE = range(6)

OK, ERR_INVALID_PE, ERR_NOT_SYMMETRIC, ERR_ALIGN, ERR_OOM, ERR_ARG = 0, -1, -2, -3, -4, -5

NP_DTYPE = {T_INT32: np.int32, T_INT64: np.int64, T_FLOAT: np.float32, T_DOUBLE: np.float64,
            T_UINT32: np.uint32, T_UINT64: np.uint64, T_INT8: np.int8, T_UINT8: np.uint8,
            T_INT16: np.int16, T_UINT16: np.uint16}


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.{os.getpid()}")
        subprocess.run(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-Wall",
                        "-shared", "-fPIC", "-o", str(tmp), str(_SRC)], check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(str(_LIB))
        vp, sz, i, u64 = C.c_void_p, C.c_size_t, C.c_int, C.c_uint64
        L.oracle_create.restype = vp
        L.oracle_create.argtypes = [i, sz]
        L.oracle_destroy.restype = None
        L.oracle_destroy.argtypes = [vp]
        L.oracle_ptr.restype = vp
        L.oracle_ptr.argtypes = [vp, sz, sz, i]
        L.oracle_malloc.argtypes = [vp, sz, sz, C.POINTER(sz)]
        L.oracle_reset_allocator.restype = None
        L.oracle_reset_allocator.argtypes = [vp]
        L.oracle_putmem.argtypes = [vp, i, sz, vp, sz, i]
        L.oracle_getmem.argtypes = [vp, i, vp, sz, sz, i]
        L.oracle_iput.argtypes = [vp, i, sz, vp, sz, sz, sz, sz, i]
        L.oracle_iget.argtypes = [vp, i, vp, sz, sz, sz, sz, sz, i]
        L.oracle_collectmem.argtypes = [vp, i, i, i, sz, sz, vp]
        L.oracle_alltoallmem.argtypes = [vp, i, i, i, sz, sz, sz]
        L.oracle_p.argtypes = [vp, sz, vp, sz, i]
        L.oracle_g.argtypes = [vp, vp, sz, sz, i]
        L.oracle_putmem_signal.argtypes = [vp, i, sz, vp, sz, sz, u64, i, i]
        L.oracle_test.argtypes = [vp, i, sz, i, u64]
        L.oracle_atomic.argtypes = [vp, i, i, sz, u64, u64, i, C.POINTER(u64)]
        L.oracle_int64_fetch_add_batch.argtypes = [vp, sz, vp, vp, vp, sz]
        L.oracle_int64_compare_swap_batch.argtypes = [vp, sz, vp, vp, vp, vp, sz]
        L.oracle_broadcastmem.argtypes = [vp, i, i, i, sz, sz, sz, i, i]
        L.oracle_fcollectmem.argtypes = [vp, i, i, i, sz, sz, sz]
        L.oracle_reduce.argtypes = [vp, i, i, i, sz, sz, sz, i, i]
        L.oracle_jacobi.argtypes = [vp, vp, sz, sz, i, C.POINTER(C.c_double)]
        L.oracle_jacobi_strip_rows.argtypes = [sz, i, i, C.POINTER(sz), C.POINTER(sz)]
        L.oracle_jacobi_scatter.argtypes = [vp, sz, vp, sz, sz]
        L.oracle_jacobi_gather.argtypes = [vp, sz, vp, sz, sz]
        L.oracle_jacobi_strips.argtypes = [vp, sz, sz, sz, sz, sz, i, C.POINTER(C.c_double)]
        L.oracle_jacobi_cell.argtypes = [vp, sz, sz, sz, sz, sz, sz, i, sz, sz,
                                         C.POINTER(C.c_double)]
        _lib = L
    return _lib


class OracleError(RuntimeError):
    def __init__(self, code: int):
        super().__init__(f"oracle error {code}")
        self.code = code


def _chk(rc: int) -> None:
    if rc != 0:
        raise OracleError(rc)


def _addr(a) -> int:
    """Raw address of a contiguous numpy array / bytes-like, or pass an int through."""
    if isinstance(a, int):
        return a
    if isinstance(a, np.ndarray):
        assert a.flags["C_CONTIGUOUS"]
        return a.ctypes.data
    raise TypeError(type(a))


class Oracle:
    """``npes`` sequential PEs, each with a ``heap_bytes`` symmetric heap (zero-filled)."""

    WORLD = None  # filled per instance: (0, 1, npes)

    def __init__(self, npes: int, heap_bytes: int):
        self.L = lib()
        self.h = self.L.oracle_create(npes, heap_bytes)
        if not self.h:
            raise MemoryError("oracle_create")
        self.npes, self.heap_bytes = npes, heap_bytes
        self.world = (0, 1, npes)

    def close(self):
        if self.h:
            self.L.oracle_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- memory ------------------------------------------------------------
    def malloc(self, size: int, align: int = 256) -> int:
        off = C.c_size_t()
        _chk(self.L.oracle_malloc(self.h, size, align, C.byref(off)))
        return off.value

    def reset_allocator(self):
        self.L.oracle_reset_allocator(self.h)

    def ptr(self, off: int, n: int, pe: int) -> int:
        p = self.L.oracle_ptr(self.h, off, n, pe)
        if not p:
            raise OracleError(ERR_NOT_SYMMETRIC)
        return p

    def view(self, off: int, n: int, pe: int, dtype=np.uint8) -> np.ndarray:
        """numpy view (no copy) of n bytes of PE ``pe``'s heap at ``off``."""
        p = self.ptr(off, n, pe)
        buf = (C.c_ubyte * n).from_address(p)
        return np.frombuffer(buf, dtype=dtype)

    # -- RMA -----------------------------------------------------------------
    def putmem(self, my_pe, dest_off, src, n, pe):
        _chk(self.L.oracle_putmem(self.h, my_pe, dest_off, _addr(src), n, pe))

    def getmem(self, my_pe, dest, src_off, n, pe):
        _chk(self.L.oracle_getmem(self.h, my_pe, _addr(dest), src_off, n, pe))

    def iput(self, my_pe, dest_off, src, dst, sst, nelems, esize, pe):
        _chk(self.L.oracle_iput(self.h, my_pe, dest_off, _addr(src), dst, sst, nelems, esize, pe))

    def iget(self, my_pe, dest, src_off, dst, sst, nelems, esize, pe):
        _chk(self.L.oracle_iget(self.h, my_pe, _addr(dest), src_off, dst, sst, nelems, esize, pe))

    def p(self, dest_off, value: np.generic | np.ndarray, pe):
        v = np.ascontiguousarray(value).reshape(1)
        _chk(self.L.oracle_p(self.h, dest_off, v.ctypes.data, v.itemsize, pe))

    def g(self, src_off, dtype, pe):
        out = np.zeros(1, dtype=dtype)
        _chk(self.L.oracle_g(self.h, out.ctypes.data, src_off, out.itemsize, pe))
        return out[0]

    def putmem_signal(self, my_pe, dest_off, src, n, sig_off, signal, sig_op, pe):
        _chk(self.L.oracle_putmem_signal(self.h, my_pe, dest_off, _addr(src), n, sig_off,
                                         signal & (2**64 - 1), sig_op, pe))

    def test(self, my_pe, ivar_off, cmp, value) -> bool:
        rc = self.L.oracle_test(self.h, my_pe, ivar_off, cmp, value & (2**64 - 1))
        if rc < 0:
            raise OracleError(rc)
        return bool(rc)

    # -- AMO -----------------------------------------------------------------
    def atomic(self, op, width, target_off, operand, cond, pe) -> int:
        old = C.c_uint64()
        m = 2**64 - 1
        _chk(self.L.oracle_atomic(self.h, op, width, target_off, operand & m, cond & m, pe,
                                  C.byref(old)))
        return old.value

    def fetch_add_batch(self, table_off, word: np.ndarray, inc: np.ndarray) -> np.ndarray:
        assert word.dtype == np.int32 and inc.dtype == np.int64
        fetched = np.empty(len(word), dtype=np.int64)
        _chk(self.L.oracle_int64_fetch_add_batch(self.h, table_off, _addr(word), _addr(inc),
                                                 _addr(fetched), len(word)))
        return fetched

    def compare_swap_batch(self, table_off, word, cond, value) -> np.ndarray:
        assert word.dtype == np.int32 and cond.dtype == np.int64 and value.dtype == np.int64
        fetched = np.empty(len(word), dtype=np.int64)
        _chk(self.L.oracle_int64_compare_swap_batch(self.h, table_off, _addr(word), _addr(cond),
                                                    _addr(value), _addr(fetched), len(word)))
        return fetched

    # -- collectives ---------------------------------------------------------
    def broadcastmem(self, team, dest_off, src_off, n, root, root_writes_dest=True):
        _chk(self.L.oracle_broadcastmem(self.h, *team, dest_off, src_off, n, root,
                                        int(root_writes_dest)))

    def fcollectmem(self, team, dest_off, src_off, n):
        _chk(self.L.oracle_fcollectmem(self.h, *team, dest_off, src_off, n))

    def collectmem(self, team, dest_off, src_off, nbytes):
        sizes = np.ascontiguousarray(nbytes, dtype=np.uint64)
        assert len(sizes) == team[2]
        _chk(self.L.oracle_collectmem(self.h, *team, dest_off, src_off, sizes.ctypes.data))

    def alltoallmem(self, team, dest_off, src_off, n):
        _chk(self.L.oracle_alltoallmem(self.h, *team, dest_off, src_off, n))

    def reduce(self, team, dest_off, src_off, nreduce, op, dtype):
        _chk(self.L.oracle_reduce(self.h, *team, dest_off, src_off, nreduce, op, dtype))

    # -- Jacobi --------------------------------------------------------------
    def jacobi_strip_rows(self, ny, pe):
        first, rows = C.c_size_t(), C.c_size_t()
        _chk(self.L.oracle_jacobi_strip_rows(ny, self.npes, pe, C.byref(first), C.byref(rows)))
        return first.value, rows.value

    def jacobi_scatter(self, buf_off, grid: np.ndarray):
        ny, nx = grid.shape
        _chk(self.L.oracle_jacobi_scatter(self.h, buf_off, _addr(grid), ny, nx))

    def jacobi_gather(self, buf_off, ny, nx) -> np.ndarray:
        grid = np.zeros((ny, nx), dtype=np.float64)
        _chk(self.L.oracle_jacobi_gather(self.h, buf_off, _addr(grid), ny, nx))
        return grid

    def jacobi_strips(self, buf0_off, buf1_off, sig_off, ny, nx, iters) -> float:
        res = C.c_double()
        _chk(self.L.oracle_jacobi_strips(self.h, buf0_off, buf1_off, sig_off, ny, nx, iters,
                                         C.byref(res)))
        return res.value


def jacobi(grid: np.ndarray, iters: int):
    """Full-grid Jacobi: returns (final grid, squared L2 norm of the last update)."""
    u = np.array(grid, dtype=np.float64, order="C", copy=True)
    scratch = np.empty_like(u)
    res = C.c_double()
    _chk(lib().oracle_jacobi(_addr(u), _addr(scratch), u.shape[0], u.shape[1], iters,
                             C.byref(res)))
    return u, res.value


def jacobi_cell(window: np.ndarray, i0: int, j0: int, ny: int, nx: int, iters: int, ci: int,
                cj: int) -> float:
    """Exact value of cell (ci, cj) after ``iters`` sweeps from a window of the initial grid."""
    w = np.ascontiguousarray(window, dtype=np.float64)
    out = C.c_double()
    _chk(lib().oracle_jacobi_cell(_addr(w), w.shape[0], w.shape[1], i0, j0, ny, nx, iters, ci, cj,
                                  C.byref(out)))
    return out.value
