"""Pins for the CPU oracle's collectives: closed forms on PE-indexed patterns,
numpy library reductions, P = 1 special cases, planted-mistake sensitivity."""
import functools
import math

import numpy as np
import pytest

import oracle as orc
from oracle import Oracle
from paper_2409_20476_b200 import inputs

NPT = {orc.T_INT32: np.int32, orc.T_INT64: np.int64, orc.T_FLOAT: np.float32,
       orc.T_DOUBLE: np.float64}


def put_src(o, off, arrs):
    for p, a in enumerate(arrs):
        o.view(off, a.nbytes, p, a.dtype)[:] = a


@pytest.mark.parametrize("P", [1, 2, 4, 12])
@pytest.mark.parametrize("dtype", [orc.T_INT32, orc.T_INT64, orc.T_FLOAT, orc.T_DOUBLE])
def test_reduce_closed_forms(P, dtype):
    """src@p[j] = K*p + j  =>  sum = K*P(P-1)/2 + P*j, max = K(P-1)+j, min = j."""
    n, K = 37, 1000
    npd = NPT[dtype]
    o = Oracle(P, 4096)
    j = np.arange(n)
    put_src(o, 0, [(K * p + j).astype(npd) for p in range(P)])
    for op, exp in ((orc.R_SUM, K * P * (P - 1) // 2 + P * j), (orc.R_MAX, K * (P - 1) + j),
                    (orc.R_MIN, j)):
        o.reduce(o.world, 1024, 0, n, op, dtype)
        for q in range(P):  # every PE holds the result
            assert np.array_equal(o.view(1024, n * np.dtype(npd).itemsize, q, npd),
                                  exp.astype(npd)), (op, q)
    # prod with src@p[j] = p + 1 is P!
    put_src(o, 0, [np.full(n, p + 1, dtype=npd) for p in range(P)])
    o.reduce(o.world, 1024, 0, n, orc.R_PROD, dtype)
    assert np.all(o.view(1024, n * np.dtype(npd).itemsize, P - 1, npd) == math.factorial(P))


def test_reduce_int_wraps_like_numpy():
    P, n = 12, 1000
    o = Oracle(P, 1 << 16)
    src = [inputs.int64_values(2, p, n) for p in range(P)]
    put_src(o, 0, src)
    o.reduce(o.world, 8192, 0, n, orc.R_PROD, orc.T_INT64)
    with np.errstate(over="ignore"):
        exp = np.prod(np.stack(src), axis=0)               # int64 product wraps mod 2^64
    assert np.array_equal(o.view(8192, 8 * n, 3, np.int64), exp)
    big = [np.full(n, 2**31 - 1 - p, dtype=np.int32) for p in range(P)]
    put_src(o, 0, big)
    o.reduce(o.world, 8192, 0, n, orc.R_SUM, orc.T_INT32)
    assert np.array_equal(o.view(8192, 4 * n, 0, np.int32), np.sum(np.stack(big), axis=0,
                                                                    dtype=np.int32))
    # bitwise operators against numpy's
    o.reduce(o.world, 8192, 0, n, orc.R_XOR, orc.T_INT32)
    assert np.array_equal(o.view(8192, 4 * n, 0, np.int32),
                          np.bitwise_xor.reduce(np.stack(big), axis=0))


@pytest.mark.parametrize("dtype", [orc.T_FLOAT, orc.T_DOUBLE])
def test_reduce_float_is_left_fold_in_pe_order(dtype):
    """A float sum over PEs equals numpy's elementwise adds applied in PE order (0 ulp),
    and differs from the reversed order on some element (so the order is really pinned)."""
    P, n = 12, 4096
    npd = NPT[dtype]
    o = Oracle(P, 1 << 17)
    src = [inputs.normal_values(2, p, n, npd) for p in range(P)]
    put_src(o, 0, src)
    for op, ufunc in ((orc.R_SUM, np.add), (orc.R_PROD, np.multiply), (orc.R_MAX, np.maximum),
                      (orc.R_MIN, np.minimum)):
        o.reduce(o.world, 1 << 16, 0, n, op, dtype)
        exp = functools.reduce(ufunc, src)
        got = o.view(1 << 16, n * np.dtype(npd).itemsize, 5, npd)
        assert got.tobytes() == exp.tobytes(), op
    o.reduce(o.world, 1 << 16, 0, n, orc.R_SUM, dtype)
    rev = functools.reduce(np.add, src[::-1])
    assert o.view(1 << 16, n * np.dtype(npd).itemsize, 0, npd).tobytes() != rev.tobytes()


def test_reduce_float_signed_zero_and_ties():
    """max/min keep the left operand unless the right is strictly greater/smaller."""
    o = Oracle(2, 256)
    o.view(0, 8, 0, np.float32)[:] = [0.0, -0.0]
    o.view(0, 8, 1, np.float32)[:] = [-0.0, 0.0]
    o.reduce(o.world, 64, 0, 2, orc.R_MAX, orc.T_FLOAT)
    got = o.view(64, 8, 0, np.float32)
    assert not np.signbit(got[0]) and np.signbit(got[1])
    o.reduce(o.world, 64, 0, 2, orc.R_MIN, orc.T_FLOAT)
    got = o.view(64, 8, 1, np.float32)
    assert not np.signbit(got[0]) and np.signbit(got[1])


def test_reduce_single_pe_is_copy_and_team_subset():
    o = Oracle(6, 4096)
    src = [inputs.int64_values(2, p, 50) for p in range(6)]
    put_src(o, 0, src)
    o.reduce((3, 1, 1), 2048, 0, 50, orc.R_SUM, orc.T_INT64)     # P = 1: a copy
    assert np.array_equal(o.view(2048, 400, 3, np.int64), src[3])
    # strided team {1, 3, 5}: only its members read and written
    o.reduce((1, 2, 3), 1024, 0, 50, orc.R_SUM, orc.T_INT64)
    exp = src[1] + src[3] + src[5]
    for q in (1, 3, 5):
        assert np.array_equal(o.view(1024, 400, q, np.int64), exp)
    for q in (0, 2, 4):
        assert not o.view(1024, 400, q).any()
    with pytest.raises(orc.OracleError):
        o.reduce((1, 2, 4), 1024, 0, 50, orc.R_SUM, orc.T_INT64)  # PE 7 does not exist


def test_reduce_uses_snapshot_when_in_place():
    o = Oracle(3, 1024)
    src = [np.arange(10, dtype=np.int32) * (p + 1) for p in range(3)]
    put_src(o, 0, src)
    o.reduce(o.world, 0, 0, 10, orc.R_SUM, orc.T_INT32)
    for q in range(3):
        assert np.array_equal(o.view(0, 40, q, np.int32), np.arange(10) * 6)


@pytest.mark.parametrize("P", [1, 3, 12])
def test_fcollect_closed_form(P):
    """src@p[k] = K*p + k  =>  dest[j] = K*(j div n) + (j mod n) on every PE."""
    n, K = 23, 100
    o = Oracle(P, 8192)
    put_src(o, 0, [(K * p + np.arange(n)).astype(np.int32) for p in range(P)])
    o.fcollectmem(o.world, 2048, 0, 4 * n)
    j = np.arange(P * n)
    exp = (K * (j // n) + j % n).astype(np.int32)
    for q in range(P):
        assert np.array_equal(o.view(2048, 4 * n * P, q, np.int32), exp)
        assert np.array_equal(o.view(0, 4 * n, q, np.int32), (K * q + np.arange(n)))  # src intact
    # equals numpy.concatenate of the sources (library routine)
    src = [inputs.byte_payload(2, p, 77) for p in range(P)]
    put_src(o, 0, src)
    o.fcollectmem(o.world, 2048, 0, 77)
    assert np.array_equal(o.view(2048, 77 * P, P - 1), np.concatenate(src))


def test_broadcast_both_root_readings_and_team():
    P, n = 5, 64
    o = Oracle(P, 1024)
    src = [inputs.byte_payload(2, p, n) for p in range(P)]
    put_src(o, 0, src)
    o.broadcastmem(o.world, 512, 0, n, 2, root_writes_dest=True)
    for q in range(P):
        assert np.array_equal(o.view(512, n, q), src[2])
    for q in range(P):
        o.view(512, n, q)[:] = 0
    o.broadcastmem(o.world, 512, 0, n, 2, root_writes_dest=False)
    for q in range(P):
        assert np.array_equal(o.view(512, n, q), src[2] if q != 2 else np.zeros(n, np.uint8))
    # root is a TEAM index: team {1,3}, root 1 -> PE 3
    for q in range(P):
        o.view(512, n, q)[:] = 0
    o.broadcastmem((1, 2, 2), 512, 0, n, 1)
    assert np.array_equal(o.view(512, n, 1), src[3]) and np.array_equal(o.view(512, n, 3), src[3])
    assert not o.view(512, n, 0).any() and not o.view(512, n, 2).any()
    with pytest.raises(orc.OracleError):
        o.broadcastmem(o.world, 1000, 0, n, 0)               # dest leaves the heap
