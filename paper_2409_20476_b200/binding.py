"""ctypes binding of the C-ABI library ``libishmem.so`` -- argument marshalling only.

Every function of ``include/ishmem.h`` is available under its own name.  Pointer
arguments accept an ``int`` device address, a ``torch.Tensor`` (its ``data_ptr()``), a
contiguous ``numpy`` array (HOST memory, for the parameters documented as host
memory) or ``None``.  Functions returning ``int`` status raise :class:`IshmemError` on a
negative status and return ``None`` otherwise; pointer-returning functions return an
``int`` address (0 = NULL).  There is no CPU path: if the library has not been built
the first call raises.
"""
from __future__ import annotations

import ctypes as C
import os
from pathlib import Path

# Device code that waits for the host proxy (ishmemx_proxy_start) needs the proxy's copy-engine
# streams to make progress while the waiting kernel runs.  CUDA maps streams onto a small number
# of hardware queues (8 unless told otherwise); work queued behind the waiting kernel on a stream
# that shares a queue with a proxy stream then sits in front of the proxy's copy and the wait
# can only end by its time limit.  32 queues give every stream of this library its own.  The
# variable is read when the CUDA context is created, so it only helps if this module is
# imported before the first CUDA call of the process; a value set by the user is kept.
os.environ.setdefault("CUDA_DEVICE_MAX_CONNECTIONS", "32")

import numpy as np

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libishmem.so"

# ---- constants of ishmem.h -------------------------------------------------------------
ISHMEM_MAX_PES = 64
(ISHMEM_OK, ISHMEM_ERR_INVALID_PE, ISHMEM_ERR_NOT_SYMMETRIC, ISHMEM_ERR_ALIGN, ISHMEM_ERR_OOM,
 ISHMEM_ERR_TIMEOUT, ISHMEM_ERR_NOT_CORESIDENT, ISHMEM_ERR_CUDA, ISHMEM_ERR_ARG,
 ISHMEM_ERR_NOT_INITIALIZED) = 0, -1, -2, -3, -4, -5, -6, -7, -8, -9
ISHMEM_TEAM_WORLD, ISHMEM_TEAM_SHARED, ISHMEM_TEAM_INVALID = 0, 1, -1
ISHMEM_SIGNAL_SET, ISHMEM_SIGNAL_ADD = 0, 1
ISHMEM_CMP_EQ, ISHMEM_CMP_NE, ISHMEM_CMP_GT, ISHMEM_CMP_GE, ISHMEM_CMP_LT, ISHMEM_CMP_LE = range(6)
(ISHMEMX_WORK_ITEM, ISHMEMX_SUB_GROUP, ISHMEMX_WORK_GROUP, ISHMEMX_WORK_GROUP_BULK,
 ISHMEMX_WORK_GROUP_ENGINE) = range(5)
(ISHMEM_OP_SUM, ISHMEM_OP_MAX, ISHMEM_OP_MIN, ISHMEM_OP_PROD, ISHMEM_OP_AND, ISHMEM_OP_OR,
 ISHMEM_OP_XOR) = range(7)
(ISHMEM_T_INT32, ISHMEM_T_INT64, ISHMEM_T_FLOAT, ISHMEM_T_DOUBLE, ISHMEM_T_UINT32,
 ISHMEM_T_UINT64, ISHMEM_T_INT8, ISHMEM_T_UINT8, ISHMEM_T_INT16, ISHMEM_T_UINT16) = range(10)
ISHMEMX_REDUCE_AUTO, ISHMEMX_REDUCE_DUPLICATED, ISHMEMX_REDUCE_SPLIT = range(3)
(ISHMEMX_OPT_JACOBI_SPLIT, ISHMEMX_OPT_JACOBI_FUSE, ISHMEMX_OPT_JACOBI_WIDE, ISHMEMX_OPT_REDUCE_BULK,
 ISHMEMX_OPT_BULK_SMEM, ISHMEMX_OPT_PUSH_SHAPE) = range(6)
SIZE_MAX = 2**64 - 1


class IshmemError(RuntimeError):
    def __init__(self, code: int, name: str):
        self.code = code
        msg = _lib.ishmem_strerror(code).decode() if _lib is not None else str(code)
        if code == ISHMEM_ERR_CUDA and _lib is not None:
            msg += ": " + _lib.ishmemx_last_cuda_error().decode()
        super().__init__(f"{name} failed: {msg} ({code})")


class _Ptr:
    """ctypes parameter type accepting ints, tensors, numpy arrays and None."""

    @classmethod
    def from_param(cls, v):
        if v is None:
            return C.c_void_p(0)
        if isinstance(v, int):
            return C.c_void_p(v)
        if hasattr(v, "data_ptr"):
            return C.c_void_p(v.data_ptr())
        if isinstance(v, np.ndarray):
            if not v.flags["C_CONTIGUOUS"]:
                raise ValueError("numpy argument must be C-contiguous")
            return C.c_void_p(v.ctypes.data)
        if isinstance(v, C.c_void_p):
            return v
        raise TypeError(f"cannot pass {type(v).__name__} as a pointer")


_CT = {"i": C.c_int, "z": C.c_size_t, "p": _Ptr, "u64": C.c_uint64, "i64": C.c_int64,
       "u32": C.c_uint32, "i32": C.c_int32, "u8": C.c_uint8, "f": C.c_float, "d": C.c_double,
       "l": C.c_long}

_RMA_TYPES = {"float": "f", "double": "d", "int": "i", "long": "l", "int32": "i32", "int64": "i64",
              "uint8": "u8", "uint32": "u32", "uint64": "u64"}
_AMO_TYPES = {"int32": "i32", "int64": "i64", "uint32": "u32", "uint64": "u64"}
_REDUCE_ARITH = ["int32", "int64", "uint32", "uint64", "float", "double", "int8", "uint8", "int16", "uint16"]
_REDUCE_BITS = ["int32", "int64", "uint32", "uint64", "int8", "uint8", "int16", "uint16"]


def _signatures() -> dict[str, tuple[str, list[str]]]:
    """name -> (return kind, argument kinds); 'status' = int status, 'ptr', 'int', 'size', 'str'."""
    S: dict[str, tuple[str, list[str]]] = {
        "ishmem_init": ("status", ["i", "z"]),
        "ishmemx_init_external": ("status", ["i", "z", "p"]),
        "ishmem_finalize": ("status", []),
        "ishmem_n_pes": ("int", []),
        "ishmemx_heap_bytes": ("size", []),
        "ishmemx_ctx": ("ptr", ["i"]),
        "ishmemx_set_stream": ("status", ["i", "p"]),
        "ishmemx_get_stream": ("ptr", ["i"]),
        "ishmem_strerror": ("str", ["i"]),
        "ishmemx_last_cuda_error": ("str", []),
        "ishmemx_status": ("int", ["i"]),
        "ishmemx_set_wait_limit_ns": ("status", ["u64"]),
        "ishmemx_set_option": ("status", ["i", "i64"]),
        "ishmemx_get_option": ("i64", ["i"]),
        "ishmemx_launch_count": ("u64", []),
        "ishmem_malloc": ("ptr", ["z"]),
        "ishmem_calloc": ("ptr", ["z", "z"]),
        "ishmem_align": ("ptr", ["z", "z"]),
        "ishmem_free": ("status", ["p"]),
        "ishmem_ptr": ("ptr", ["p", "i"]),
        "ishmemx_heap_write": ("status", ["i", "p", "p", "z"]),
        "ishmemx_heap_read": ("status", ["i", "p", "p", "z"]),
        "ishmem_putmem": ("status", ["i", "p", "p", "z", "i"]),
        "ishmem_getmem": ("status", ["i", "p", "p", "z", "i"]),
        "ishmem_putmem_nbi": ("status", ["i", "p", "p", "z", "i"]),
        "ishmem_getmem_nbi": ("status", ["i", "p", "p", "z", "i"]),
        "ishmemx_putmem_on_device": ("status", ["i", "p", "p", "z", "i", "i", "i", "i"]),
        "ishmemx_getmem_on_device": ("status", ["i", "p", "p", "z", "i", "i", "i", "i"]),
        "ishmemx_putmem_copy_engine": ("status", ["i", "p", "p", "z", "i"]),
        "ishmemx_getmem_copy_engine": ("status", ["i", "p", "p", "z", "i"]),
        "ishmemx_putmem_spmd": ("status", ["p", "p", "z", "i", "i", "i", "i"]),
        "ishmemx_getmem_spmd": ("status", ["p", "p", "z", "i", "i", "i", "i"]),
        "ishmemx_putmem_spmd_copy_engine": ("status", ["p", "p", "z", "i"]),
        "ishmemx_set_cutover": ("status", ["i", "z"]),
        "ishmemx_get_cutover": ("size", ["i"]),
        "ishmemx_tune_cutover": ("status", ["i", "i", "z", "p"]),
        "ishmem_putmem_signal": ("status", ["i", "p", "p", "z", "p", "u64", "i", "i"]),
        "ishmem_uint64_wait_until": ("status", ["i", "p", "i", "u64"]),
        "ishmemx_iputmem": ("status", ["i", "p", "p", "z", "z", "z", "z", "i"]),
        "ishmemx_igetmem": ("status", ["i", "p", "p", "z", "z", "z", "z", "i"]),
        "ishmem_uint64_test": ("status", ["i", "p", "i", "u64", "p"]),
        "ishmem_uint64_wait_until_all": ("status", ["i", "p", "z", "p", "i", "u64"]),
        "ishmem_uint64_wait_until_any": ("status", ["i", "p", "z", "p", "i", "u64", "p"]),
        "ishmem_uint64_wait_until_some": ("status", ["i", "p", "z", "p", "p", "i", "u64", "p"]),
        "ishmem_collectmem": ("status", ["i", "p", "p", "p"]),
        "ishmem_alltoallmem": ("status", ["i", "p", "p", "z"]),
        "ishmem_fence": ("status", ["i"]),
        "ishmem_quiet": ("status", ["i"]),
        "ishmem_team_sync": ("status", ["i"]),
        "ishmem_sync_all": ("status", []),
        "ishmem_barrier_all": ("status", []),
        "ishmem_team_split_strided": ("int", ["i", "i", "i", "i"]),
        "ishmem_team_split_2d": ("status", ["i", "i", "i", "p", "p"]),
        "ishmem_team_destroy": ("status", ["i"]),
        "ishmem_team_n_pes": ("int", ["i"]),
        "ishmem_team_my_pe": ("int", ["i", "i"]),
        "ishmem_team_translate_pe": ("int", ["i", "i", "i"]),
        "ishmem_info_get_version": ("void", ["p", "p"]),
        "ishmem_info_get_name": ("void", ["p"]),
        "ishmemx_int64_atomic_fetch_add_batch": ("status", ["p", "p", "p", "p", "z", "i", "i"]),
        "ishmemx_int64_atomic_compare_swap_batch": ("status", ["p", "p", "p", "p", "p", "z", "i", "i"]),
        "ishmem_broadcastmem": ("status", ["i", "p", "p", "z", "i"]),
        "ishmemx_set_bcast_root_dest": ("status", ["i"]),
        "ishmem_fcollectmem": ("status", ["i", "p", "p", "z"]),
        "ishmemx_reduce": ("status", ["i", "p", "p", "z", "i", "i", "i"]),
        "ishmemx_set_collective_geometry": ("status", ["i", "i"]),
        "ishmemx_collective_on_device": ("status", ["i", "i", "p", "p", "z", "i", "i", "i", "i", "i"]),
        "ishmemx_pingpong": ("status", ["i", "i", "p", "p", "z", "i", "i", "p", "p"]),
        "ishmemx_pingpong_phases": ("status", ["i", "i", "p", "p", "z", "i", "i", "i", "p"]),
        "ishmemx_proxy_start": ("status", []),
        "ishmemx_proxy_stop": ("status", []),
        "ishmemx_proxy_stats": ("status", ["p", "p", "p"]),
        "ishmemx_ring_benchmark": ("status", ["i", "i", "i", "i", "p", "p"]),
        "ishmemx_rma_latency": ("status", ["i", "p", "p", "z", "i", "i", "i", "i", "i", "p"]),
        "ishmemx_jacobi": ("status", ["p", "p", "p", "z", "z", "i", "i", "i", "i", "p"]),
        "ishmemx_jacobi_launch_depths": ("int", ["i", "i", "p", "i"]),
        "ishmemx_jacobi_noalloc": ("status", ["p", "p", "p", "z", "z", "i", "i", "i", "i", "p"]),
        "ishmemx_host_put_ring": ("status", ["p", "p", "p", "p", "z", "i", "i", "i", "i"]),
    }
    for name, t in _RMA_TYPES.items():
        for op in ("put", "get", "put_nbi", "get_nbi"):
            S[f"ishmem_{name}_{op}"] = ("status", ["i", "p", "p", "z", "i"])
        S[f"ishmem_{name}_broadcast"] = ("status", ["i", "p", "p", "z", "i"])
        S[f"ishmem_{name}_fcollect"] = ("status", ["i", "p", "p", "z"])
        S[f"ishmem_{name}_collect"] = ("status", ["i", "p", "p", "p"])
        S[f"ishmem_{name}_alltoall"] = ("status", ["i", "p", "p", "z"])
        S[f"ishmem_{name}_iput"] = ("status", ["i", "p", "p", "z", "z", "z", "i"])
        S[f"ishmem_{name}_iget"] = ("status", ["i", "p", "p", "z", "z", "z", "i"])
        S[f"ishmem_{name}_p"] = ("status", ["i", "p", t, "i"])
        S[f"ishmem_{name}_g"] = ("status", ["i", "p", "p", "i"])
    for name, t in _AMO_TYPES.items():
        pre = f"ishmem_{name}_atomic_"
        S[pre + "add"] = ("status", ["i", "p", t, "i"])
        S[pre + "inc"] = ("status", ["i", "p", "i"])
        S[pre + "set"] = ("status", ["i", "p", t, "i"])
        for op in ("and", "or", "xor"):
            S[pre + op] = ("status", ["i", "p", t, "i"])
        S[pre + "fetch"] = ("status", ["i", "p", "p", "i"])
        S[pre + "fetch_inc"] = ("status", ["i", "p", "p", "i"])
        for op in ("fetch_add", "swap", "fetch_and", "fetch_or", "fetch_xor"):
            S[pre + op] = ("status", ["i", "p", "p", t, "i"])
        S[pre + "compare_swap"] = ("status", ["i", "p", "p", t, t, "i"])
    for name in _REDUCE_ARITH:
        for op in ("sum", "max", "min", "prod"):
            S[f"ishmem_{name}_{op}_reduce"] = ("status", ["i", "p", "p", "z"])
    for name in _REDUCE_BITS:
        for op in ("and", "or", "xor"):
            S[f"ishmem_{name}_{op}_reduce"] = ("status", ["i", "p", "p", "z"])
    return S


SIGNATURES = _signatures()
_lib = None


def _status_check(name):
    def check(result, func, args):
        if result < 0:
            raise IshmemError(result, name)
        return None
    return check


def lib() -> C.CDLL:
    """Loads ``libishmem.so`` (raises if it has not been built) and types every entry point."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                               "`python -m paper_2409_20476_b200.build` (there is no CPU fallback)")
        L = C.CDLL(str(LIB_PATH))
        for name, (ret, args) in SIGNATURES.items():
            f = getattr(L, name)
            f.argtypes = [_CT[a] for a in args]
            if ret == "status":
                f.restype = C.c_int
                f.errcheck = _status_check(name)
            elif ret == "void":
                f.restype = None
            elif ret == "int":
                f.restype = C.c_int
            elif ret == "ptr":
                f.restype = C.c_void_p
                f.errcheck = lambda r, fn, a: int(r or 0)
            elif ret == "size":
                f.restype = C.c_size_t
            elif ret == "u64":
                f.restype = C.c_uint64
            elif ret == "i64":
                f.restype = C.c_int64
            elif ret == "str":
                f.restype = C.c_char_p
        _lib = L
    return _lib


def __getattr__(name: str):
    if name in SIGNATURES:
        return getattr(lib(), name)
    raise AttributeError(name)


def strerror(code: int) -> str:
    return lib().ishmem_strerror(code).decode()
