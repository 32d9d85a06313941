"""A user's own kernel, compiled separately against include/ishmem_device.cuh, calls the device
API with contexts obtained from ishmemx_ctx: work-group put, in-kernel barrier, remote atomic,
strided put and device-resident reduce -- checked against the oracle."""
import ctypes as C
from pathlib import Path

import numpy as np
import pytest
import torch

import oracle as orc
from paper_2409_20476_b200 import binding as B
from paper_2409_20476_b200 import build as libbuild
from paper_2409_20476_b200 import inputs
from tests.gpu_util import Session, heaps_equal

pytestmark = pytest.mark.gpu


def test_user_kernel_against_the_public_device_header():
    so = libbuild.build_user_kernel_example()
    user = C.CDLL(str(so))
    user.user_launch_ring_step.restype = C.c_int
    user.user_launch_ring_step.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p,
                                           C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    npes, n, nred = 6, 40_000, 3001
    with Session(npes, 1 << 20) as s:
        src, dst, cnt = s.malloc(n), s.malloc(2 * n), s.malloc(64)
        rs, rd = s.malloc(4 * nred), s.malloc(4 * nred)
        for p in range(npes):
            src.fill(p, inputs.byte_payload(inputs.SEED_C2, 90 + p, n))
            rs.fill(p, inputs.int32_reduce_values(inputs.SEED_C1, 90 + p, nred))
        s.sync()
        stream = torch.cuda.Stream()
        rc = user.user_launch_ring_step(B.ishmemx_ctx(0), npes, dst.addr, src.addr, n, cnt.addr, rd.addr, rs.addr, nred,
                                        stream.cuda_stream)
        assert rc == 0
        o = s.oracle
        for p in range(npes):
            o.putmem(p, dst.ooff, o.ptr(src.ooff, n, p), n, (p + 1) % npes)
        for p in range(npes):
            o.atomic(orc.A_FETCH_ADD, 8, cnt.ooff, p + 1, 0, 0)
        for p in range(npes):
            o.iput(p, dst.ooff + n, o.ptr(dst.ooff, n, p), 1, 2, n // 8, 4, (p + npes - 1) % npes)
        o.reduce(o.world, rd.ooff, rs.ooff, nred, orc.R_SUM, orc.T_INT32)
        heaps_equal(s, "user kernel")
        assert cnt.read(0, np.int64)[0] == npes * (npes + 1) // 2
        assert s.status() == 0
