"""Degenerate and extreme shapes against the oracle: one PE, the maximum number of PEs,
zero-length operations, strided teams, sizes around the kernels' internal thresholds."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2409_20476_b200 import binding as B
from paper_2409_20476_b200 import inputs
from tests.gpu_util import Session, heaps_equal

pytestmark = pytest.mark.gpu
W = B.ISHMEM_TEAM_WORLD


def run_everything(s, npes, n, team=None, oteam=None):
    """one pass of every collective and a put/get ring of n bytes on both sides"""
    o = s.oracle
    team = W if team is None else team
    oteam = o.world if oteam is None else oteam
    P = oteam[2]
    src, dst = s.malloc(max(n * P, 64)), s.malloc(max(n * P * P, 64))
    for p in range(npes):
        src.fill(p, inputs.byte_payload(inputs.SEED_C2, 200 + p, max(n * P, 64)))
    for p in range(npes):
        t = (p + 1) % npes
        B.ishmem_putmem(p, dst.addr, src.addr, n, t)
        o.putmem(p, dst.ooff, o.ptr(src.ooff, n, p), n, t)
    B.ishmem_barrier_all()
    for p in range(npes):
        t = (p + npes - 1) % npes
        B.ishmem_getmem(p, dst.addr + n, src.addr, n, t)
        o.getmem(p, o.ptr(dst.ooff + n, n, p), src.ooff, n, t)
    B.ishmem_barrier_all()
    heaps_equal(s, f"put/get ring npes={npes} n={n}")
    B.ishmem_broadcastmem(team, dst.addr, src.addr, n, P - 1)
    o.broadcastmem(oteam, dst.ooff, src.ooff, n, P - 1)
    heaps_equal(s, "broadcast")
    B.ishmem_fcollectmem(team, dst.addr, src.addr, n)
    o.fcollectmem(oteam, dst.ooff, src.ooff, n)
    heaps_equal(s, "fcollect")
    B.ishmem_alltoallmem(team, dst.addr, src.addr, n)
    o.alltoallmem(oteam, dst.ooff, src.ooff, n)
    heaps_equal(s, "alltoall")
    sizes = [(n * (i % 3)) // 2 for i in range(P)]
    B.ishmem_collectmem(team, dst.addr, src.addr, np.array(sizes, dtype=np.uint64))
    o.collectmem(oteam, dst.ooff, src.ooff, sizes)
    heaps_equal(s, "collect")
    for alg in (B.ISHMEMX_REDUCE_SPLIT, B.ISHMEMX_REDUCE_DUPLICATED):
        B.ishmemx_reduce(team, dst.addr, src.addr, n // 8, B.ISHMEM_OP_XOR, B.ISHMEM_T_UINT64, alg)
        o.reduce(oteam, dst.ooff, src.ooff, n // 8, orc.R_XOR, orc.T_UINT64)
        # (the payload is random bytes: as floats they would contain NaNs, whose payloads are outside
        # the bit-exact contract, so the arithmetic fold here is the wrapping int32 sum)
        B.ishmemx_reduce(team, dst.addr + 8 * (n // 8 + 1), src.addr, n // 4, B.ISHMEM_OP_SUM, B.ISHMEM_T_INT32, alg)
        o.reduce(oteam, dst.ooff + 8 * (n // 8 + 1), src.ooff, n // 4, orc.R_SUM, orc.T_INT32)
        heaps_equal(s, f"reduce alg={alg}")
    B.ishmem_team_sync(team)
    assert s.status() == 0


@pytest.mark.parametrize("n", [0, 8, 4104])
def test_a_single_pe_is_a_valid_job(n):
    """P = 1: every collective degenerates to a local copy (reduce of one source = that source)."""
    with Session(1, 1 << 18) as s:
        run_everything(s, 1, n)


@pytest.mark.parametrize("n", [0, 16, 1032])
def test_the_maximum_number_of_pes(n):
    """64 PEs (ISHMEM_MAX_PES): translation tables, push sync and the collectives at full width."""
    npes = B.ISHMEM_MAX_PES
    with Session(npes, (1 << 16) + n * npes * npes * 2) as s:
        run_everything(s, npes, n)
        with pytest.raises(B.IshmemError) as e:
            B.ishmem_putmem(0, s.malloc(64).addr, s.malloc(64).addr, 8, npes)
        assert e.value.code == B.ISHMEM_ERR_INVALID_PE


def test_more_pes_than_the_library_supports_is_refused():
    heap = torch.zeros(65 * 4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.IshmemError) as e:
        B.ishmemx_init_external(B.ISHMEM_MAX_PES + 1, 4096, heap.data_ptr())
    assert e.value.code == B.ISHMEM_ERR_ARG


def test_strided_teams_only_touch_their_members():
    npes = 12
    with Session(npes, 1 << 20) as s:
        team = B.ishmem_team_split_strided(W, 2, 4, 3)                 # PEs 2, 6, 10
        assert B.ishmem_team_n_pes(team) == 3
        run_everything(s, npes, 2056, team, (2, 4, 3))
        sub = B.ishmem_team_split_strided(team, 1, 1, 2)                # PEs 6, 10 of the parent
        src, dst = s.malloc(4096), s.malloc(8192)
        for p in range(npes):
            src.fill(p, inputs.byte_payload(inputs.SEED_C3, 300 + p, 4096))
        B.ishmem_fcollectmem(sub, dst.addr, src.addr, 3000)
        s.oracle.fcollectmem((6, 4, 2), dst.ooff, src.ooff, 3000)
        heaps_equal(s, "team of a team")
        assert [B.ishmem_team_my_pe(team, p) for p in (2, 6, 10, 3, 11)] == [0, 1, 2, -1, -1]
        assert [B.ishmem_team_my_pe(sub, p) for p in (2, 6, 10)] == [-1, 0, 1]
        assert B.ishmem_team_translate_pe(sub, 1, team) == 2 and B.ishmem_team_translate_pe(team, 0, sub) == -1
        assert B.ishmem_team_translate_pe(team, 2, W) == 10 and B.ishmem_team_translate_pe(W, 7, team) == -1
        major, minor, name = np.zeros(1, np.int32), np.zeros(1, np.int32), np.zeros(64, np.uint8)
        B.ishmem_info_get_version(major, minor)
        B.ishmem_info_get_name(name)
        assert (major[0], minor[0]) == (1, 5) and bytes(name).split(b"\0")[0].startswith(b"ishmem")
        B.ishmem_team_destroy(sub)
        B.ishmem_team_destroy(team)
        assert B.ishmem_team_split_strided(W, 0, 5, 4) == B.ISHMEM_TEAM_INVALID     # 0, 5, 10, 15: outside
        assert s.status() == 0


@pytest.mark.parametrize("n", [16383, 16384, 16385, (1 << 20) - 1, (1 << 20) + 16, (4 << 20) + 1])
def test_sizes_around_the_internal_thresholds(n):
    """bulk-ring minimum (16 KiB), the 1 MiB push threshold, the 4 MiB host cutover"""
    npes = 4
    with Session(npes, 3 * n + (1 << 20)) as s:
        src, dst = s.malloc(n + 32), s.malloc(2 * n + 64)
        for p in range(npes):
            src.fill(p, inputs.byte_payload(inputs.SEED_C2, 400 + p, n + 32))
        for p in range(npes):
            B.ishmem_putmem(p, dst.addr + 1, src.addr + 1, n, (p + 1) % npes)               # default cutover
            s.oracle.putmem(p, dst.ooff + 1, s.oracle.ptr(src.ooff + 1, n, p), n, (p + 1) % npes)
        B.ishmemx_putmem_spmd(dst.addr + n + 16, src.addr + 16, n, 2, B.ISHMEMX_WORK_GROUP_BULK, 256, 2)
        for p in range(npes):
            s.oracle.putmem(p, dst.ooff + n + 16, s.oracle.ptr(src.ooff + 16, n, p), n, (p + 2) % npes)
        B.ishmem_barrier_all()
        heaps_equal(s, f"puts n={n}")
        B.ishmem_broadcastmem(W, dst.addr, src.addr, n, 1)
        s.oracle.broadcastmem(s.oracle.world, dst.ooff, src.ooff, n, 1)
        heaps_equal(s, f"broadcast n={n}")
        assert s.status() == 0


def test_two_dimensional_team_split():
    """12 PEs as a 3 x 4 grid (xrange 4), and a ragged 5-column split of the same 12."""
    npes = 12
    with Session(npes, 1 << 18) as s:
        src, dst = s.malloc(4096), s.malloc(16384)
        for p in range(npes):
            src.fill(p, inputs.byte_payload(inputs.SEED_C3, 600 + p, 4096))
        tx, ty = np.zeros(1, np.int32), np.zeros(1, np.int32)
        B.ishmem_team_split_2d(W, 4, 6, tx, ty)                 # PE 6 = (x 2, y 1)
        assert [B.ishmem_team_my_pe(int(tx[0]), p) for p in range(npes)] == [-1] * 4 + [0, 1, 2, 3] + [-1] * 4
        assert [B.ishmem_team_my_pe(int(ty[0]), p) for p in range(npes)] == [-1, -1, 0, -1, -1, -1, 1, -1, -1, -1, 2, -1]
        B.ishmem_fcollectmem(int(tx[0]), dst.addr, src.addr, 1000)
        s.oracle.fcollectmem((4, 1, 4), dst.ooff, src.ooff, 1000)
        B.ishmemx_reduce(int(ty[0]), dst.addr + 8192, src.addr, 500, B.ISHMEM_OP_XOR, B.ISHMEM_T_UINT64, B.ISHMEMX_REDUCE_AUTO)
        s.oracle.reduce((2, 4, 3), dst.ooff + 8192, src.ooff, 500, orc.R_XOR, orc.T_UINT64)
        heaps_equal(s, "2-D teams")
        B.ishmem_team_destroy(int(tx[0]))
        B.ishmem_team_destroy(int(ty[0]))
        B.ishmem_team_split_2d(W, 5, 11, tx, ty)                # ragged: rows 0-4, 5-9, 10-11; PE 11 = (x 1, y 2)
        assert B.ishmem_team_n_pes(int(tx[0])) == 2 and B.ishmem_team_n_pes(int(ty[0])) == 3
        assert B.ishmem_team_my_pe(int(tx[0]), 10) == 0 and B.ishmem_team_my_pe(int(ty[0]), 6) == 1
        with pytest.raises(B.IshmemError):
            B.ishmem_team_split_2d(W, 0, 0, tx, ty)
        assert s.status() == 0


def test_calloc_is_ordered_before_any_pes_next_operation():
    """calloc clears every PE's copy as one team operation: a put or an atomic that another PE
    issues right after it, with no barrier in between, lands on zeroed memory and stays.  The
    region is large, dirty beforehand and the puts hit its far end, where a clearing that
    another PE's stream still had in flight would wipe them out."""
    npes, n = 4, 96 << 20
    with Session(npes, n + (1 << 20), with_oracle=False) as s:
        for rep in range(3):
            s.heap.fill_(0xA5)
            torch.cuda.synchronize()
            p = B.ishmem_calloc(n // 8, 8)
            assert p
            tail = p + n - 4096
            for me in range(npes):
                t = (me + 1) % npes
                B.ishmem_uint64_p(me, tail + 8 * me, 1000 + me, t)             # a scalar put into the neighbour
                B.ishmem_uint64_atomic_add(me, tail + 2048, 1, (me + 2) % npes)  # and an atomic two PEs on
            B.ishmem_barrier_all()
            s.sync()
            off = p - s.base
            for q in range(npes):
                got = s.heap[q * s.heap_bytes + off:q * s.heap_bytes + off + n].view(torch.int64)
                exp_nonzero = {(n - 4096) // 8 + (q - 1) % npes: 1000 + (q - 1) % npes, (n - 4096 + 2048) // 8: 1}
                nz = torch.nonzero(got).flatten().cpu().tolist()
                assert sorted(nz) == sorted(exp_nonzero), (rep, q, nz)
                for k, v in exp_nonzero.items():
                    assert int(got[k]) == v, (rep, q, k)
            B.ishmem_free(p)
        assert s.status() == 0
