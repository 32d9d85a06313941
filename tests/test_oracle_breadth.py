"""Pins of the oracle's strided RMA, collect, alltoall and 8/16-bit reductions against what
numpy and the definitions fix (no GPU, nothing of the CUDA path)."""
import numpy as np
import pytest

import oracle as orc


@pytest.fixture
def o():
    x = orc.Oracle(5, 1 << 14)
    yield x
    x.close()


def fill(o, off, n, seed):
    r = np.random.default_rng(seed)
    for p in range(o.npes):
        o.view(off, n, p)[:] = r.integers(0, 256, n, dtype=np.uint8)


@pytest.mark.parametrize("esize", [1, 2, 4, 8, 16])
@pytest.mark.parametrize("dst,sst,nelems", [(1, 1, 17), (3, 1, 9), (1, 4, 11), (2, 5, 7), (7, 3, 1), (4, 4, 0)])
def test_iput_iget_equal_numpy_strided_slices(o, esize, dst, sst, nelems):
    src_off, dst_off, span = 0, 4096, 2048
    fill(o, 0, 8192, esize * 100 + dst * 10 + sst)
    before = [o.view(0, 8192, p).copy() for p in range(o.npes)]
    local = before[1][src_off:src_off + span].copy()
    o.iput(1, dst_off, local, dst, sst, nelems, esize, 3)
    exp = before[3].copy()
    e = exp[dst_off:dst_off + span].reshape(-1, esize)
    e[:nelems * dst:dst][:nelems] = local.reshape(-1, esize)[:nelems * sst:sst][:nelems]
    assert np.array_equal(o.view(0, 8192, 3), exp)
    for p in (0, 1, 2, 4):
        assert np.array_equal(o.view(0, 8192, p), before[p])          # nobody else touched
    # iget: the mirror image, into private memory
    out = np.full(span, 0xEE, dtype=np.uint8)
    o.iget(2, out, dst_off, dst, sst, nelems, esize, 3)
    ref = np.full(span, 0xEE, dtype=np.uint8).reshape(-1, esize)
    ref[:nelems * dst:dst][:nelems] = o.view(dst_off, span, 3).reshape(-1, esize)[:nelems * sst:sst][:nelems]
    assert np.array_equal(out, ref.ravel())


def test_iput_with_unit_strides_is_put_and_bad_arguments_are_refused(o):
    fill(o, 0, 4096, 1)
    a = orc.Oracle(5, 1 << 14)
    try:
        for p in range(5):
            a.view(0, 4096, p)[:] = o.view(0, 4096, p)
        src = o.view(100, 300, 0).copy()
        o.iput(0, 1000, src, 1, 1, 75, 4, 2)
        a.putmem(0, 1000, src, 300, 2)
        assert np.array_equal(o.view(0, 4096, 2), a.view(0, 4096, 2))
    finally:
        a.close()
    with pytest.raises(orc.OracleError):
        o.iput(0, 0, src, 0, 1, 3, 4, 1)                     # stride 0
    with pytest.raises(orc.OracleError):
        o.iput(0, (1 << 14) - 16, src, 3, 1, 5, 4, 1)        # runs off the heap
    with pytest.raises(orc.OracleError):
        o.iget(0, src, 0, 1, 1, 3, 4, 9)                     # no such PE


def test_collect_is_the_concatenation_in_team_order(o):
    sizes = [7, 0, 300, 1, 45]
    fill(o, 0, 512, 3)
    parts = [o.view(0, sizes[p], p).copy() for p in range(5)]
    o.collectmem(o.world, 2048, 0, sizes)
    exp = np.concatenate(parts)
    for q in range(5):
        assert np.array_equal(o.view(2048, exp.size, q), exp)
        assert not o.view(2048 + exp.size, 64, q).any()             # nothing past the end
    # equal sizes: the same as fcollect
    o.collectmem(o.world, 4096, 0, [33] * 5)
    o.fcollectmem(o.world, 8192, 0, 33)
    assert np.array_equal(o.view(4096, 165, 2), o.view(8192, 165, 2))
    # a strided sub-team {1, 3}
    o.collectmem((1, 2, 2), 12000, 0, [5, 9])
    assert np.array_equal(o.view(12000, 14, 3), np.concatenate([parts[1][:0], o.view(0, 5, 1), o.view(0, 9, 3)]))
    assert not o.view(12000, 14, 0).any() and not o.view(12000, 14, 2).any()


def test_alltoall_is_a_block_transpose_and_an_involution(o):
    n, P = 24, 5
    fill(o, 0, n * P, 4)
    src = np.stack([o.view(0, n * P, p).reshape(P, n).copy() for p in range(P)])     # [i, q, k]
    o.alltoallmem(o.world, 4096, 0, n)
    got = np.stack([o.view(4096, n * P, q).reshape(P, n) for q in range(P)])          # [q, i, k]
    assert np.array_equal(got, src.transpose(1, 0, 2))
    o.alltoallmem(o.world, 8192, 4096, n)                      # applying it twice gives the input back
    for p in range(P):
        assert np.array_equal(o.view(8192, n * P, p), o.view(0, n * P, p))
    # closed form on a PE-indexed pattern: src@i[q*n + k] = 1000*i + 10*q + k
    for i in range(P):
        o.view(0, 4 * n * P, i, np.int32)[:] = (1000 * i + 10 * np.arange(P)[:, None] + np.arange(n)[None, :]).ravel()
    o.alltoallmem(o.world, 4096, 0, 4 * n)
    for q in range(P):
        exp = (1000 * np.arange(P)[:, None] + 10 * q + np.arange(n)[None, :]).ravel()
        assert np.array_equal(o.view(4096, 4 * n * P, q, np.int32), exp)


@pytest.mark.parametrize("dt,npd", [(orc.T_INT8, np.int8), (orc.T_UINT8, np.uint8), (orc.T_INT16, np.int16),
                                    (orc.T_UINT16, np.uint16)])
def test_narrow_integer_reductions_wrap_like_numpy(o, dt, npd):
    n = 257
    r = np.random.default_rng(5)
    info = np.iinfo(npd)
    vals = r.integers(info.min, info.max + 1, size=(5, n), dtype=np.int64).astype(npd)
    for p in range(5):
        o.view(0, n * vals.itemsize, p, npd)[:] = vals[p]
    ref = {orc.R_SUM: np.add.reduce(vals, axis=0, dtype=npd), orc.R_PROD: np.multiply.reduce(vals, axis=0, dtype=npd),
           orc.R_MAX: vals.max(axis=0), orc.R_MIN: vals.min(axis=0), orc.R_AND: np.bitwise_and.reduce(vals, axis=0),
           orc.R_OR: np.bitwise_or.reduce(vals, axis=0), orc.R_XOR: np.bitwise_xor.reduce(vals, axis=0)}
    for op, exp in ref.items():
        o.reduce(o.world, 4096, 0, n, op, dt)
        for q in (0, 4):
            assert np.array_equal(o.view(4096, n * vals.itemsize, q, npd), exp), op
    # closed form: sum of p+1 over 5 PEs = 15; product = 120 (wraps for 8-bit signed: 120 fits)
    for p in range(5):
        o.view(0, n * vals.itemsize, p, npd)[:] = p + 1
    o.reduce(o.world, 4096, 0, n, orc.R_SUM, dt)
    assert (o.view(4096, n * vals.itemsize, 1, npd) == 15).all()
    o.reduce(o.world, 4096, 0, n, orc.R_PROD, dt)
    assert (o.view(4096, n * vals.itemsize, 1, npd) == 120).all()
