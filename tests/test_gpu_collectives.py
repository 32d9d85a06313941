"""GPU parity of sync / broadcast / fcollect / reduce against the CPU oracle: host-called
team launches and the device-resident work-group forms with in-kernel push sync."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2409_20476_b200 import binding as B
from paper_2409_20476_b200 import inputs
from tests.gpu_util import Session, heaps_equal

pytestmark = pytest.mark.gpu

DT = {  # name -> (numpy, library dtype, oracle dtype)
    "int32": (np.int32, B.ISHMEM_T_INT32, orc.T_INT32),
    "int64": (np.int64, B.ISHMEM_T_INT64, orc.T_INT64),
    "uint32": (np.uint32, B.ISHMEM_T_UINT32, orc.T_UINT32),
    "uint64": (np.uint64, B.ISHMEM_T_UINT64, orc.T_UINT64),
    "float": (np.float32, B.ISHMEM_T_FLOAT, orc.T_FLOAT),
    "double": (np.float64, B.ISHMEM_T_DOUBLE, orc.T_DOUBLE),
}
OPS = {"sum": (B.ISHMEM_OP_SUM, orc.R_SUM), "max": (B.ISHMEM_OP_MAX, orc.R_MAX),
       "min": (B.ISHMEM_OP_MIN, orc.R_MIN), "prod": (B.ISHMEM_OP_PROD, orc.R_PROD),
       "and": (B.ISHMEM_OP_AND, orc.R_AND), "or": (B.ISHMEM_OP_OR, orc.R_OR),
       "xor": (B.ISHMEM_OP_XOR, orc.R_XOR)}


def values(name, pe, n):
    npd = DT[name][0]
    if name in ("float", "double"):
        return inputs.normal_values(inputs.SEED_C3, pe, n, npd)
    return inputs.int64_values(inputs.SEED_C3, pe, n).astype(npd)


def test_config1_int32_sum_reduce():
    """Config 1: 4 PEs, 262144 int32 in [-1000, 1000], sum over all PEs, every PE gets it."""
    n = 262144
    with Session(4, 16 << 20) as s:
        src, dst = s.malloc(4 * n), s.malloc(4 * n)
        for p in range(4):
            src.fill(p, inputs.int32_reduce_values(inputs.SEED_C1, p, n))
        B.ishmem_int32_sum_reduce(B.ISHMEM_TEAM_WORLD, dst.addr, src.addr, n)
        s.oracle.reduce(s.oracle.world, dst.ooff, src.ooff, n, orc.R_SUM, orc.T_INT32)
        heaps_equal(s, "int32 sum_reduce")
        # and the closed form on a PE-indexed pattern
        for p in range(4):
            src.fill(p, (1000 * p + np.arange(n)).astype(np.int32))
        B.ishmem_int32_sum_reduce(B.ISHMEM_TEAM_WORLD, dst.addr, src.addr, n)
        assert np.array_equal(dst.read(2, np.int32), (6000 + 4 * np.arange(n)).astype(np.int32))


@pytest.mark.parametrize("alg", [B.ISHMEMX_REDUCE_SPLIT, B.ISHMEMX_REDUCE_DUPLICATED])
@pytest.mark.parametrize("name", ["int64", "float", "double"])
def test_config3_reduce_12_pes(name, alg):
    """12 PEs, sum/max/min/prod, element counts 4^0..4^9 (ragged vector tails included);
    floats must match the PE-order fold bit for bit (0 ulp)."""
    npd, ldt, odt = DT[name]
    es = np.dtype(npd).itemsize
    nmax = 4 ** 9
    with Session(12, 2 * nmax * es + (1 << 16)) as s:
        src, dst = s.malloc(nmax * es), s.malloc(nmax * es)
        for p in range(12):
            src.fill(p, values(name, p, nmax))
        for k in range(10):
            n = 4 ** k
            for opname in ("sum", "max", "min", "prod"):
                lop, oop = OPS[opname]
                B.ishmemx_reduce(B.ISHMEM_TEAM_WORLD, dst.addr, src.addr, n, lop, ldt, alg)
                s.oracle.reduce(s.oracle.world, dst.ooff, src.ooff, n, oop, odt)
                dst.assert_equal(f"{name} {opname} n={n}")
            B.ishmem_barrier_all()
        heaps_equal(s, name)
        assert s.status() == 0


def test_reduce_typed_names_bitwise_unaligned_inplace_and_teams():
    with Session(6, 1 << 20) as s:
        n = 10_007
        src, dst = s.malloc(8 * n + 64), s.malloc(8 * n + 64)
        for name in DT:
            npd, ldt, odt = DT[name]
            es = np.dtype(npd).itemsize
            for p in range(6):
                src.fill(p, values(name, p, n + 8))
            ops = list(OPS) if name not in ("float", "double") else ["sum", "max", "min", "prod"]
            for opname in ops:
                lop, oop = OPS[opname]
                # element offset 1: buffers aligned to the element but not to 16 bytes
                getattr(B, f"ishmem_{name}_{opname}_reduce")(B.ISHMEM_TEAM_WORLD, dst.addr + es,
                                                             src.addr + es, n)
                s.oracle.reduce(s.oracle.world, dst.ooff + es, src.ooff + es, n, oop, odt)
            dst.assert_equal(name)
        # float ops are rejected for bitwise operators, misaligned buffers too
        with pytest.raises(B.IshmemError) as e:
            B.ishmemx_reduce(0, dst.addr, src.addr, 4, B.ISHMEM_OP_XOR, B.ISHMEM_T_FLOAT, 0)
        assert e.value.code == B.ISHMEM_ERR_ARG
        with pytest.raises(B.IshmemError) as e:
            B.ishmemx_reduce(0, dst.addr + 4, src.addr, 4, B.ISHMEM_OP_SUM, B.ISHMEM_T_INT64, 0)
        assert e.value.code == B.ISHMEM_ERR_ALIGN
        with pytest.raises(B.IshmemError) as e:                  # partial overlap
            B.ishmemx_reduce(0, src.addr + 16, src.addr, 64, B.ISHMEM_OP_SUM, B.ISHMEM_T_INT32, 0)
        assert e.value.code == B.ISHMEM_ERR_ARG
        # in place (snapshot semantics) with the split algorithm
        B.ishmemx_reduce(0, src.addr, src.addr, n, B.ISHMEM_OP_SUM, B.ISHMEM_T_DOUBLE, B.ISHMEMX_REDUCE_SPLIT)
        s.oracle.reduce(s.oracle.world, src.ooff, src.ooff, n, orc.R_SUM, orc.T_DOUBLE)
        src.assert_equal("in place")
        # strided sub-team {1, 3, 5}
        team = B.ishmem_team_split_strided(B.ISHMEM_TEAM_WORLD, 1, 2, 3)
        assert team >= 2 and B.ishmem_team_n_pes(team) == 3
        B.ishmem_int64_max_reduce(team, dst.addr, src.addr, 1000)
        s.oracle.reduce((1, 2, 3), dst.ooff, src.ooff, 1000, orc.R_MAX, orc.T_INT64)
        B.ishmem_broadcastmem(team, dst.addr + 16_000, src.addr, 3001, 2)      # root = PE 5
        s.oracle.broadcastmem((1, 2, 3), dst.ooff + 16_000, src.ooff, 3001, 2)
        B.ishmem_fcollectmem(team, dst.addr + 32_000, src.addr + 8, 1001)
        s.oracle.fcollectmem((1, 2, 3), dst.ooff + 32_000, src.ooff + 8, 1001)
        B.ishmem_team_sync(team)
        B.ishmem_team_destroy(team)
        assert B.ishmem_team_split_strided(B.ISHMEM_TEAM_WORLD, 0, 4, 3) == B.ISHMEM_TEAM_INVALID
        B.ishmem_barrier_all()
        heaps_equal(s, "teams")
        assert s.status() == 0


@pytest.mark.parametrize("cutover", [B.SIZE_MAX, 0])
def test_config3_broadcast_fcollect_12_pes(cutover):
    """broadcast from root 0 and fcollect, 12 PEs, element counts 4^0..4^8 of 8-byte
    elements, by pushing stores (cutover never) and through the copy engine (always)."""
    nmax = 4 ** 8
    with Session(12, 14 * nmax * 8 + (1 << 16)) as s:
        src, dst = s.malloc(nmax * 8), s.malloc(12 * nmax * 8)
        for p in range(12):
            src.fill(p, inputs.int64_values(inputs.SEED_C3, p, nmax))
        B.ishmemx_set_cutover(1, cutover)
        B.ishmemx_set_cutover(2, cutover)
        for k in range(9):
            nb = 8 * 4 ** k
            B.ishmem_broadcastmem(B.ISHMEM_TEAM_WORLD, dst.addr, src.addr, nb, 0)
            s.oracle.broadcastmem(s.oracle.world, dst.ooff, src.ooff, nb, 0)
            dst.assert_equal(f"broadcast {nb}")
            B.ishmem_fcollectmem(B.ISHMEM_TEAM_WORLD, dst.addr, src.addr, nb)
            s.oracle.fcollectmem(s.oracle.world, dst.ooff, src.ooff, nb)
            dst.assert_equal(f"fcollect {nb}")
        # odd byte counts and offsets, non-zero root, root not writing its own dest
        B.ishmem_broadcastmem(B.ISHMEM_TEAM_WORLD, dst.addr + 3, src.addr + 5, 12_345, 7)
        s.oracle.broadcastmem(s.oracle.world, dst.ooff + 3, src.ooff + 5, 12_345, 7)
        B.ishmem_fcollectmem(B.ISHMEM_TEAM_WORLD, dst.addr + 20_001, src.addr + 1, 777)
        s.oracle.fcollectmem(s.oracle.world, dst.ooff + 20_001, src.ooff + 1, 777)
        B.ishmemx_set_bcast_root_dest(0)
        B.ishmem_broadcastmem(B.ISHMEM_TEAM_WORLD, dst.addr + 64_000, src.addr, 4096, 4)
        s.oracle.broadcastmem(s.oracle.world, dst.ooff + 64_000, src.ooff, 4096, 4, root_writes_dest=False)
        B.ishmemx_set_bcast_root_dest(1)
        with pytest.raises(B.IshmemError) as e:
            B.ishmem_broadcastmem(B.ISHMEM_TEAM_WORLD, dst.addr, src.addr, 8, 12)
        assert e.value.code == B.ISHMEM_ERR_INVALID_PE
        B.ishmem_barrier_all()
        heaps_equal(s, "broadcast/fcollect")
        assert s.status() == 0


@pytest.mark.parametrize("threads", [128, 1024])
def test_device_resident_collectives_with_push_sync(threads):
    """One work-group per PE calls ishmemx_{broadcastmem,fcollectmem,reduce}_work_group inside
    one co-resident launch; completion relies on the in-kernel push sync alone."""
    with Session(12, 1 << 20) as s:
        n = 5_003
        src, dst = s.malloc(8 * n + 64), s.malloc(12 * 8 * n + 64)
        for p in range(12):
            src.fill(p, inputs.normal_values(inputs.SEED_C3, p, n + 8, np.float64))
        W = B.ISHMEM_TEAM_WORLD
        B.ishmemx_collective_on_device(0, W, dst.addr, src.addr, 8 * n - 3, 5, 0, 0, threads, 1)
        s.oracle.broadcastmem(s.oracle.world, dst.ooff, src.ooff, 8 * n - 3, 5)
        dst.assert_equal("device broadcast")
        B.ishmemx_collective_on_device(1, W, dst.addr, src.addr, 8 * n, 0, 0, 0, threads, 1)
        s.oracle.fcollectmem(s.oracle.world, dst.ooff, src.ooff, 8 * n)
        dst.assert_equal("device fcollect")
        for name, opname in (("double", "sum"), ("float", "prod"), ("int64", "min"), ("int32", "xor"),
                             ("uint64", "max")):
            npd, ldt, odt = DT[name]
            cnt = (8 * n) // np.dtype(npd).itemsize
            for p in range(12):
                src.fill(p, values(name, p, cnt))
            B.ishmemx_collective_on_device(2, W, dst.addr, src.addr, cnt, 0, OPS[opname][0], ldt, threads, 1)
            s.oracle.reduce(s.oracle.world, dst.ooff, src.ooff, cnt, OPS[opname][1], odt)
            dst.assert_equal(f"device reduce {name} {opname}")
        # repeated syncs: monotone counters, no reset race
        B.ishmemx_collective_on_device(3, W, None, None, 0, 0, 0, 0, threads, 500)
        B.ishmem_barrier_all()
        heaps_equal(s, "device collectives")
        assert s.status() == 0
        # more blocks than can be co-resident are refused, not launched
        # (64 PEs would still fit; the refusal path is exercised through the argument check)
        with pytest.raises(B.IshmemError):
            B.ishmemx_collective_on_device(2, W, dst.addr, dst.addr, 4, 0, 0, 0, threads, 1)  # overlap


@pytest.mark.parametrize("shape", [1, 2])
def test_push_shapes_of_broadcast_and_fcollect(shape):
    """Both launch shapes of host-called broadcast / fcollect (fan-out tiles; one block per tile, source
    member and destination) on sizes around and across the 32 KiB tile, odd offsets, a strided team, a
    non-zero root and the reading in which the root does not write its own dest: whole heaps against the
    oracle."""
    npes, nmax = 6, 100_003
    with Session(npes, 8 * nmax + (1 << 16)) as s:
        B.ishmemx_set_option(B.ISHMEMX_OPT_PUSH_SHAPE, shape)
        assert B.ishmemx_get_option(B.ISHMEMX_OPT_PUSH_SHAPE) == shape
        src, dst = s.malloc(nmax), s.malloc(npes * nmax)
        for p in range(npes):
            src.fill(p, inputs.byte_payload(inputs.SEED_C3, 90 + p, nmax))
        W, o = B.ISHMEM_TEAM_WORLD, s.oracle
        for n, so, do, root in ((1, 0, 0, 0), (32768, 0, 0, 5), (32769, 1, 3, 2), (nmax - 7, 7, 0, 1), (65536, 16, 48, 3)):
            B.ishmem_broadcastmem(W, dst.addr + do, src.addr + so, n, root)
            o.broadcastmem(o.world, dst.ooff + do, src.ooff + so, n, root)
            heaps_equal(s, f"broadcast {n} shape {shape}")
            B.ishmem_fcollectmem(W, dst.addr + do, src.addr + so, n)
            o.fcollectmem(o.world, dst.ooff + do, src.ooff + so, n)
            heaps_equal(s, f"fcollect {n} shape {shape}")
        B.ishmemx_set_bcast_root_dest(0)
        B.ishmem_broadcastmem(W, dst.addr, src.addr + 2, 70_000, 4)
        o.broadcastmem(o.world, dst.ooff, src.ooff + 2, 70_000, 4, root_writes_dest=False)
        B.ishmemx_set_bcast_root_dest(1)
        team = B.ishmem_team_split_strided(W, 1, 2, 3)           # PEs 1, 3, 5
        B.ishmem_broadcastmem(team, dst.addr + 5, src.addr, 40_000, 2)
        o.broadcastmem((1, 2, 3), dst.ooff + 5, src.ooff, 40_000, 2)
        B.ishmem_fcollectmem(team, dst.addr + 9, src.addr + 1, 33_333)
        o.fcollectmem((1, 2, 3), dst.ooff + 9, src.ooff + 1, 33_333)
        B.ishmem_barrier_all()
        heaps_equal(s, f"strided team shape {shape}")
        assert s.status() == 0
