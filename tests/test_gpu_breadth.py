"""GPU parity of the wider OpenSHMEM surface: strided put/get, collect, alltoall, 8/16-bit
reductions, test and the multi-word waits -- each against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2409_20476_b200 import binding as B
from paper_2409_20476_b200 import inputs
from tests.gpu_util import Session, heaps_equal

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("es,dstr,sstr,n", [(8, 3, 2, 70_001), (4, 1, 5, 1024 * 9), (16, 2, 1, 4 * 1024 + 1), (1, 2, 2, 300_000)])
def test_strided_messages_of_many_tiles(es, dstr, sstr, n):
    """strided put and get whose elements span many 1024-element tiles of the launch and a ragged
    last tile; whole heaps against the oracle"""
    npes = 2
    span = ((n - 1) * max(dstr, sstr) + 1) * es + 64
    with Session(npes, 2 * span + (1 << 12)) as s:
        src, dst = s.malloc(span), s.malloc(span)
        for p in range(npes):
            src.fill(p, inputs.byte_payload(inputs.SEED_C2, 60 + p, span))
        B.ishmemx_iputmem(0, dst.addr + es, src.addr + 2 * es, dstr, sstr, n, es, 1)
        s.oracle.iput(0, dst.ooff + es, s.oracle.ptr(src.ooff + 2 * es, ((n - 1) * sstr + 1) * es, 0), dstr, sstr, n, es, 1)
        B.ishmem_barrier_all()
        heaps_equal(s, "iput")
        B.ishmemx_igetmem(1, src.addr, dst.addr + es, sstr, dstr, n, es, 0)      # PE 1 gathers from PE 0's dst
        s.oracle.iget(1, s.oracle.ptr(src.ooff, ((n - 1) * sstr + 1) * es, 1), dst.ooff + es, sstr, dstr, n, es, 0)
        B.ishmem_barrier_all()
        heaps_equal(s, "iget")
        assert s.status() == 0


@pytest.mark.parametrize("es", [1, 2, 4, 8, 16])
def test_strided_put_get_match_the_oracle(es):
    npes, heap = 3, 1 << 19
    with Session(npes, heap) as s:
        src, dst = s.malloc(200_000), s.malloc(200_000)
        for p in range(npes):
            src.fill(p, inputs.byte_payload(inputs.SEED_C2, 50 + p, 200_000))
        for dstr, sstr, n in ((1, 1, 17), (3, 1, 9), (1, 4, 11), (2, 5, 1000), (7, 3, 1), (4, 4, 0), (2, 3, 3500 // es)):
            so, do = 3 * es, 5 * es
            B.ishmemx_iputmem(1, dst.addr + do, src.addr + so, dstr, sstr, n, es, 2)
            sspan = ((n - 1) * sstr + 1) * es if n else 0
            s.oracle.iput(1, dst.ooff + do, s.oracle.ptr(src.ooff + so, sspan, 1), dstr, sstr, n, es, 2)
            B.ishmem_barrier_all()
            heaps_equal(s, f"iput es={es} {dstr},{sstr},{n}")
            dspan = ((n - 1) * dstr + 1) * es if n else 0
            B.ishmemx_igetmem(0, src.addr + do, dst.addr + so, dstr, sstr, n, es, 2)
            s.oracle.iget(0, s.oracle.ptr(src.ooff + do, dspan, 0), dst.ooff + so, dstr, sstr, n, es, 2)
            B.ishmem_barrier_all()
            heaps_equal(s, f"iget es={es} {dstr},{sstr},{n}")
        assert s.status() == 0


def test_strided_typed_names_and_argument_checks():
    with Session(2, 1 << 16) as s:
        a, b = s.malloc(8192), s.malloc(8192)
        a.fill(0, inputs.normal_values(inputs.SEED_C3, 0, 1024, np.float64))
        B.ishmem_double_iput(0, b.addr, a.addr, 2, 3, 100, 1)
        s.oracle.iput(0, b.ooff, s.oracle.ptr(a.ooff, 8192, 0), 2, 3, 100, 8, 1)
        B.ishmem_double_iget(1, a.addr + 8, b.addr, 1, 2, 50, 1)
        s.oracle.iget(1, s.oracle.ptr(a.ooff + 8, 400, 1), b.ooff, 1, 2, 50, 8, 1)
        B.ishmem_barrier_all()
        heaps_equal(s, "typed strided")
        for args, code in (((0, b.addr, a.addr, 0, 1, 4, 8, 1), B.ISHMEM_ERR_ARG),
                           ((0, b.addr, a.addr, 1, 1, 4, 3, 1), B.ISHMEM_ERR_ARG),
                           ((0, b.addr + 4, a.addr, 1, 1, 4, 8, 1), B.ISHMEM_ERR_ALIGN),
                           ((0, b.addr, a.addr, 4000, 1, 4000, 8, 1), B.ISHMEM_ERR_NOT_SYMMETRIC),
                           ((0, b.addr, a.addr, 1, 1, 4, 8, 5), B.ISHMEM_ERR_INVALID_PE)):
            with pytest.raises(B.IshmemError) as e:
                B.ishmemx_iputmem(*args)
            assert e.value.code == code, args
        assert s.status() == 0


def test_collect_and_alltoall_12_pes():
    npes = 12
    sizes = [7, 0, 300_001, 1, 45, 4096, 2 << 20, 16, 100_000, 3, 65_536, 999]
    total = sum(sizes)
    with Session(npes, 2 * total + (8 << 20)) as s:
        src, dst = s.malloc(max(sizes) + 4096), s.malloc(total + 64)
        for p in range(npes):
            src.fill(p, inputs.byte_payload(inputs.SEED_C3, 60 + p, max(sizes)))
        szs = np.array(sizes, dtype=np.uint64)
        B.ishmem_collectmem(B.ISHMEM_TEAM_WORLD, dst.addr, src.addr, szs)
        s.oracle.collectmem(s.oracle.world, dst.ooff, src.ooff, sizes)
        heaps_equal(s, "collect")
        team = B.ishmem_team_split_strided(B.ISHMEM_TEAM_WORLD, 1, 3, 4)          # PEs 1, 4, 7, 10
        B.ishmem_collectmem(team, dst.addr + 3, src.addr + 1, np.array([5, 70_000, 0, 33], dtype=np.uint64))
        s.oracle.collectmem((1, 3, 4), dst.ooff + 3, src.ooff + 1, [5, 70_000, 0, 33])
        heaps_equal(s, "collect on a strided team")
        for n in (1, 24, 4099, 100_000):
            B.ishmem_alltoallmem(B.ISHMEM_TEAM_WORLD, dst.addr, src.addr, n)
            s.oracle.alltoallmem(s.oracle.world, dst.ooff, src.ooff, n)
            heaps_equal(s, f"alltoall n={n}")
        B.ishmem_alltoallmem(team, dst.addr + 16, src.addr + 48, 5000)
        s.oracle.alltoallmem((1, 3, 4), dst.ooff + 16, src.ooff + 48, 5000)
        heaps_equal(s, "alltoall on a strided team")
        # device-resident form: one work-group per PE, in-kernel sync
        B.ishmemx_collective_on_device(4, B.ISHMEM_TEAM_WORLD, dst.addr, src.addr, 3001, 0, 0, 0, 256, 1)
        s.oracle.alltoallmem(s.oracle.world, dst.ooff, src.ooff, 3001)
        heaps_equal(s, "alltoall_work_group")
        # collect with the sizes exchanged inside the kernel (member i gives n * ((i mod 3) + 1) / 3 bytes), twice
        for n in (3000, 10):
            B.ishmemx_collective_on_device(5, B.ISHMEM_TEAM_WORLD, dst.addr, src.addr, n, 0, 0, 0, 128, 2)
            s.oracle.collectmem(s.oracle.world, dst.ooff, src.ooff, [n * (i % 3 + 1) // 3 for i in range(npes)])
            heaps_equal(s, f"collect_work_group n={n}")
        with pytest.raises(B.IshmemError):
            B.ishmem_alltoallmem(B.ISHMEM_TEAM_WORLD, src.addr + 8, src.addr, 64)   # overlap
        # typed names (counts in elements)
        B.ishmem_double_broadcast(B.ISHMEM_TEAM_WORLD, dst.addr, src.addr, 1000, 3)
        s.oracle.broadcastmem(s.oracle.world, dst.ooff, src.ooff, 8000, 3)
        B.ishmem_int32_fcollect(team, dst.addr, src.addr, 777)
        s.oracle.fcollectmem((1, 3, 4), dst.ooff, src.ooff, 4 * 777)
        B.ishmem_uint64_alltoall(team, dst.addr + 64, src.addr, 99)
        s.oracle.alltoallmem((1, 3, 4), dst.ooff + 64, src.ooff, 8 * 99)
        B.ishmem_float_collect(team, dst.addr + 8, src.addr + 4, np.array([3, 0, 1000, 17], dtype=np.uint64))
        s.oracle.collectmem((1, 3, 4), dst.ooff + 8, src.ooff + 4, [12, 0, 4000, 68])
        heaps_equal(s, "typed collectives")
        with pytest.raises(B.IshmemError) as e:
            B.ishmem_double_fcollect(team, dst.addr + 4, src.addr, 8)
        assert e.value.code == B.ISHMEM_ERR_ALIGN
        B.ishmem_team_destroy(team)
        assert s.status() == 0


NARROW = {"int8": (np.int8, B.ISHMEM_T_INT8, orc.T_INT8), "uint8": (np.uint8, B.ISHMEM_T_UINT8, orc.T_UINT8),
          "int16": (np.int16, B.ISHMEM_T_INT16, orc.T_INT16), "uint16": (np.uint16, B.ISHMEM_T_UINT16, orc.T_UINT16)}
OPS = [(B.ISHMEM_OP_SUM, orc.R_SUM), (B.ISHMEM_OP_MAX, orc.R_MAX), (B.ISHMEM_OP_MIN, orc.R_MIN),
       (B.ISHMEM_OP_PROD, orc.R_PROD), (B.ISHMEM_OP_AND, orc.R_AND), (B.ISHMEM_OP_OR, orc.R_OR),
       (B.ISHMEM_OP_XOR, orc.R_XOR)]


@pytest.mark.parametrize("name", list(NARROW))
def test_narrow_integer_reductions_12_pes(name):
    npd, ldt, odt = NARROW[name]
    es, npes, nmax = np.dtype(npd).itemsize, 12, 300_001
    with Session(npes, 2 * nmax * es + (1 << 16)) as s:
        src, dst = s.malloc(nmax * es), s.malloc(nmax * es)
        info = np.iinfo(npd)
        for p in range(npes):
            r = inputs.rng_for(inputs.SEED_C3, 70, p)
            src.fill(p, r.integers(info.min, info.max + 1, size=nmax, dtype=np.int64).astype(npd))
        for n in (1, 37, 5000, nmax):
            for alg in (B.ISHMEMX_REDUCE_SPLIT, B.ISHMEMX_REDUCE_DUPLICATED):
                for lop, oop in OPS:
                    B.ishmemx_reduce(B.ISHMEM_TEAM_WORLD, dst.addr, src.addr, n, lop, ldt, alg)
                    s.oracle.reduce(s.oracle.world, dst.ooff, src.ooff, n, oop, odt)
                    dst.assert_equal(f"{name} n={n} alg={alg} op={lop}")
        getattr(B, f"ishmem_{name}_sum_reduce")(B.ISHMEM_TEAM_WORLD, dst.addr + 2, src.addr + 2, 999)
        s.oracle.reduce(s.oracle.world, dst.ooff + 2, src.ooff + 2, 999, orc.R_SUM, odt)
        B.ishmemx_collective_on_device(2, B.ISHMEM_TEAM_WORLD, dst.addr, src.addr, 4097, 0, B.ISHMEM_OP_PROD, ldt, 128, 1)
        s.oracle.reduce(s.oracle.world, dst.ooff, src.ooff, 4097, orc.R_PROD, odt)
        heaps_equal(s, name)
        assert s.status() == 0


def test_test_and_multi_word_waits():
    with Session(2, 1 << 16) as s:
        iv = s.malloc(64)
        B.ishmemx_set_wait_limit_ns(50_000_000)
        res = np.zeros(1, np.int32)
        B.ishmem_uint64_p(1, iv.addr + 16, 7, 0)          # word 2 of PE 0
        B.ishmem_uint64_p(1, iv.addr + 40, 9, 0)          # word 5 of PE 0
        s.oracle.p(iv.ooff + 16, np.uint64(7), 0)
        s.oracle.p(iv.ooff + 40, np.uint64(9), 0)
        B.ishmem_barrier_all()
        for cmp_l, cmp_o in ((B.ISHMEM_CMP_EQ, orc.C_EQ), (B.ISHMEM_CMP_NE, orc.C_NE), (B.ISHMEM_CMP_GT, orc.C_GT),
                             (B.ISHMEM_CMP_GE, orc.C_GE), (B.ISHMEM_CMP_LT, orc.C_LT), (B.ISHMEM_CMP_LE, orc.C_LE)):
            for word in (0, 2, 5):
                for v in (0, 7, 8):
                    B.ishmem_uint64_test(0, iv.addr + 8 * word, cmp_l, v, res)
                    assert bool(res[0]) == s.oracle.test(0, iv.ooff + 8 * word, cmp_o, v), (cmp_l, word, v)
        idx, cnt, found = np.zeros(1, np.uint64), np.zeros(1, np.uint64), np.zeros(8, np.uint64)
        B.ishmem_uint64_wait_until_any(0, iv.addr, 8, None, B.ISHMEM_CMP_GE, 7, idx)
        assert idx[0] == 2
        B.ishmem_uint64_wait_until_any(0, iv.addr, 8, None, B.ISHMEM_CMP_GT, 7, idx)
        assert idx[0] == 5
        B.ishmem_uint64_wait_until_some(0, iv.addr, 8, found, None, B.ISHMEM_CMP_NE, 0, cnt)
        assert cnt[0] == 2 and list(found[:2]) == [2, 5]
        # the status mask takes words out of the wait: word 2 masked -> only word 5 qualifies
        mask = torch.zeros(8, dtype=torch.int32, device="cuda")
        mask[2] = 1
        torch.cuda.synchronize()
        B.ishmem_uint64_wait_until_any(0, iv.addr, 8, mask, B.ISHMEM_CMP_NE, 0, idx)
        assert idx[0] == 5
        B.ishmem_uint64_wait_until_some(0, iv.addr, 8, found, mask, B.ISHMEM_CMP_NE, 0, cnt)
        assert cnt[0] == 1 and found[0] == 5
        allbut = torch.ones(8, dtype=torch.int32, device="cuda")
        allbut[2] = allbut[5] = 0
        torch.cuda.synchronize()
        B.ishmem_uint64_wait_until_all(0, iv.addr, 8, allbut, B.ISHMEM_CMP_GE, 7)     # only words 2 and 5 count
        B.ishmem_uint64_wait_until_all(0, iv.addr, 8, None, B.ISHMEM_CMP_LE, 9)
        assert s.status() == 0
        # nothing on PE 1 satisfies these: bounded waits give up and say so
        with pytest.raises(B.IshmemError) as e:
            B.ishmem_uint64_wait_until_any(1, iv.addr, 8, None, B.ISHMEM_CMP_NE, 0, idx)
        assert e.value.code == B.ISHMEM_ERR_TIMEOUT
        assert s.status() == B.ISHMEM_ERR_TIMEOUT
        B.ishmem_uint64_wait_until_all(0, iv.addr, 8, None, B.ISHMEM_CMP_NE, 0)
        assert s.status() == B.ISHMEM_ERR_TIMEOUT
        with pytest.raises(B.IshmemError):
            B.ishmem_uint64_wait_until_all(0, iv.addr, 257, None, B.ISHMEM_CMP_NE, 0)
