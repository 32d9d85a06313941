"""Parity at the full benchmark sizes, in the launch configurations the benchmark times.

The CPU oracle cannot process these sizes whole in reasonable time, so each test checks
(a) a property that holds at any size over the WHOLE output (a put delivers the sender's
bytes; every PE holds the same reduce result; ...), computed on the device from the inputs,
and (b) sampled windows -- message head and tail, slice and tile boundaries, random offsets
-- against the oracle run on exactly those windows of the regenerated inputs."""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

import oracle as orc
from paper_2409_20476_b200 import binding as B
from paper_2409_20476_b200 import inputs
from tests.gpu_util import Session

pytestmark = pytest.mark.gpu
MiB = 1 << 20
POOL = ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1))


def fill_full(sym, kind, seed, nelems, npes):
    """Every PE's copy of `sym` <- block_values(kind, seed, pe, 0, nelems), generated in
    chunks by a thread pool (the generator releases the GIL) and uploaded chunk by chunk."""
    chunk = 8 * inputs.BLOCK_ELEMS
    es = np.dtype({"u8": np.uint8, "f32": np.float32, "f64": np.float64, "i64": np.int64}[kind]).itemsize
    jobs = [(p, c) for p in range(npes) for c in range(0, nelems, chunk)]

    def gen(job):
        p, c = job
        return p, c, inputs.block_values(kind, seed, p, c, min(chunk, nelems - c))

    for p, c, v in POOL.map(gen, jobs):
        sym.gpu(p)[c * es:c * es + v.nbytes].copy_(torch.from_numpy(v.view(np.uint8)))
    torch.cuda.synchronize()          # torch's stream is not ordered with the library's streams


def windows(n, width, rng, extra=()):
    """start offsets of sampled windows of `width` units in [0, n): both ends, the given
    extra points (clamped), and random ones"""
    pts = {0, max(0, n - width)}
    for e in extra:
        for d in (-width // 2, 0):
            pts.add(int(min(max(0, e + d), max(0, n - width))))
    for o in rng.integers(0, max(1, n - width), size=24):
        pts.add(int(o))
    return sorted(pts)


@pytest.mark.parametrize("level,threads,groups", [("tiled", 256, 0), ("bulk", 256, 37), ("ldst", 512, 74)])
def test_config2_put_get_256mib_ring_and_all_pairs(level, threads, groups):
    """Config 2 at its largest size: 8 PEs x 512 MiB heap, 256 MiB uint8 messages, ring and the
    7 all-pairs rounds, in the geometry the benchmark launches (groups = 0: one tile of threads x 128
    bytes per block) and in the two resident-grid alternatives."""
    npes, heap, n = 8, 512 * MiB, 256 * MiB
    lv = {"tiled": B.ISHMEMX_WORK_GROUP, "bulk": B.ISHMEMX_WORK_GROUP_BULK, "ldst": B.ISHMEMX_WORK_GROUP}[level]
    rng = np.random.default_rng(7)
    with Session(npes, heap, with_oracle=False) as s:
        src, dst = s.malloc(n), s.malloc(n)
        fill_full(src, "u8", inputs.SEED_C2, n, npes)
        nslices = groups if groups else n // (threads * 128)
        per = -(-n // nslices)
        per = (per + 127) // 128 * 128
        offs = windows(n, 4096, rng, extra=[per * g for g in (1, 2, nslices // 2, nslices - 1)])
        for shift in range(1, npes):
            B.ishmemx_putmem_spmd(dst.addr, src.addr, n, shift, lv, threads, groups)
            s.sync()
            for p in range(npes):
                assert torch.equal(dst.gpu((p + shift) % npes), src.gpu(p)), (shift, p)
            if shift == 1:
                o = orc.Oracle(npes, 1 << 14)
                try:
                    for off in offs:
                        for p in range(npes):
                            o.view(0, 4096, p)[:] = inputs.block_values("u8", inputs.SEED_C2, p, off, 4096)
                        for p in range(npes):
                            o.putmem(p, 8192, o.ptr(0, 4096, p), 4096, (p + 1) % npes)
                        for q in range(npes):
                            got = dst.gpu(q)[off:off + 4096].cpu().numpy()
                            assert np.array_equal(got, o.view(8192, 4096, q)), (off, q)
                finally:
                    o.close()
        # get: PE p fetches src@(p+3) into its dst
        for p in range(npes):
            dst.gpu(p).zero_()
        s.sync()
        B.ishmemx_getmem_spmd(dst.addr, src.addr, n, 3, lv, threads, groups)
        s.sync()
        for p in range(npes):
            assert torch.equal(dst.gpu(p), src.gpu((p + 3) % npes)), p
        # the copy-engine path on the same pattern
        for p in range(npes):
            dst.gpu(p).zero_()
        s.sync()
        B.ishmemx_putmem_spmd_copy_engine(dst.addr, src.addr, n, 1)
        s.sync()
        for p in range(npes):
            assert torch.equal(dst.gpu((p + 1) % npes), src.gpu(p)), p
        assert s.status() == 0


KIND = {"f32": (np.float32, B.ISHMEM_T_FLOAT, orc.T_FLOAT), "f64": (np.float64, B.ISHMEM_T_DOUBLE, orc.T_DOUBLE),
        "i64": (np.int64, B.ISHMEM_T_INT64, orc.T_INT64)}
OPS = [(B.ISHMEM_OP_SUM, orc.R_SUM), (B.ISHMEM_OP_MAX, orc.R_MAX), (B.ISHMEM_OP_MIN, orc.R_MIN),
       (B.ISHMEM_OP_PROD, orc.R_PROD)]


@pytest.mark.parametrize("kind,nelems", [("f32", 4 ** 13), ("f64", 4 ** 12), ("i64", 4 ** 12)])
def test_config3_reduce_large_12_pes(kind, nelems):
    """Config 3 at large counts: 12 PEs, sum/max/min/prod.  Whole output: all PEs hold
    identical results.  Windows: the PE-order fold of the oracle, bit for bit (0 ulp)."""
    npd, ldt, odt = KIND[kind]
    es, npes, W = np.dtype(npd).itemsize, 12, 1024
    rng = np.random.default_rng(8)
    with Session(npes, 2 * nelems * es + MiB, with_oracle=False) as s:
        src, dst = s.malloc(nelems * es), s.malloc(nelems * es)
        fill_full(src, kind, inputs.SEED_C3, nelems, npes)
        offs = windows(nelems, W, rng, extra=[nelems // 12 * k for k in (1, 5, 11)] + [nelems // 2])
        o = orc.Oracle(npes, 1 << 15)
        try:
            for lop, oop in OPS:
                B.ishmemx_reduce(B.ISHMEM_TEAM_WORLD, dst.addr, src.addr, nelems, lop, ldt, B.ISHMEMX_REDUCE_AUTO)
                s.sync()
                for q in range(1, npes):
                    assert torch.equal(dst.gpu(q), dst.gpu(0)), (lop, q)
                for off in offs:
                    for p in range(npes):
                        o.view(0, W * es, p, npd)[:] = inputs.block_values(kind, inputs.SEED_C3, p, off, W)
                    o.reduce(o.world, 16384, 0, W, oop, odt)
                    got = dst.gpu(3)[off * es:(off + W) * es].cpu().numpy()
                    assert got.tobytes() == o.view(16384, W * es, 3).tobytes(), (lop, off)
        finally:
            o.close()
        assert s.status() == 0


def test_config3_broadcast_fcollect_large_12_pes():
    """Config 3: broadcast of 64 Mi float32 (256 MiB) from root 0 and fcollect of 16 Mi
    float32 per PE (768 MiB gathered on every PE), 12 PEs."""
    npes, nb, nf = 12, 4 * 4 ** 13, 4 * 4 ** 12
    rng = np.random.default_rng(9)
    with Session(npes, nb + npes * nf + MiB, with_oracle=False) as s:
        src, dst = s.malloc(nb), s.malloc(npes * nf)
        fill_full(src, "f32", inputs.SEED_C3, nb // 4, npes)
        B.ishmem_broadcastmem(B.ISHMEM_TEAM_WORLD, dst.addr, src.addr, nb, 0)
        s.sync()
        for q in range(npes):
            assert torch.equal(dst.gpu(q)[:nb], src.gpu(0)), q
        o = orc.Oracle(npes, 1 << 17)
        try:
            W = 4096
            for off in windows(nb, W, rng):
                off &= ~3
                for p in range(npes):
                    o.view(0, W, p)[:] = inputs.block_values("f32", inputs.SEED_C3, p, off // 4, W // 4).view(np.uint8)
                o.broadcastmem(o.world, 4096, 0, W, 0)
                for q in (0, 7, 11):
                    assert np.array_equal(dst.gpu(q)[off:off + W].cpu().numpy(), o.view(4096, W, q)), (off, q)
            B.ishmem_fcollectmem(B.ISHMEM_TEAM_WORLD, dst.addr, src.addr, nf)
            s.sync()
            for q in range(npes):
                for i in range(npes):
                    assert torch.equal(dst.gpu(q)[i * nf:(i + 1) * nf], src.gpu(i)[:nf]), (q, i)
            for off in windows(nf, W, rng):
                off &= ~3
                for p in range(npes):
                    o.view(0, W, p)[:] = inputs.block_values("f32", inputs.SEED_C3, p, off // 4, W // 4).view(np.uint8)
                o.fcollectmem(o.world, 4096, 0, W)
                exp = o.view(4096, npes * W, 5).reshape(npes, W)
                for i in range(npes):
                    got = dst.gpu(5)[i * nf + off:i * nf + off + W].cpu().numpy()
                    assert np.array_equal(got, exp[i]), (off, i)
        finally:
            o.close()
        assert s.status() == 0


def test_config5_jacobi_16384_200_iterations_sampled_cells():
    """Config 5 at full size: 16384 x 16384 float64, 12 row strips, 200 sweeps with in-kernel
    put_signal halos.  Sampled cells -- corners, edges, strip boundaries, interior -- are
    compared bit for bit with the oracle's dependency-cone evaluation from the initial grid."""
    npes, n, iters = 12, 16384, 200
    rows_max = -(-n // npes)
    nbytes = (rows_max + 2) * n * 8
    nblk = n // 1024
    grid = np.empty((n, n))

    def gen(b):
        grid[b * 1024:(b + 1) * 1024] = inputs.jacobi_grid_block(inputs.SEED_C5, n, n, b)

    list(POOL.map(gen, range(nblk)))
    base, extra = divmod(n, npes)
    firsts = [p * base + min(p, extra) for p in range(npes + 1)]
    with Session(npes, 2 * nbytes + MiB, with_oracle=False) as s:
        b0, b1, sig = s.malloc(nbytes), s.malloc(nbytes), s.malloc(64)
        for p in range(npes):
            rows = firsts[p + 1] - firsts[p]
            b0.gpu(p)[n * 8:(rows + 1) * n * 8].copy_(torch.from_numpy(grid[firsts[p]:firsts[p + 1]].view(np.uint8).ravel()))
        s.sync()
        for p in range(npes):
            sig.fill(p, np.zeros(64, np.uint8))
        s.sync()
        B.ishmemx_jacobi(b0.addr, b1.addr, sig.addr, n, n, iters, 1, 12, 0, None)
        assert s.status() == 0
        rng = np.random.default_rng(10)
        cells = [(1, 1), (n - 2, n - 2), (1, n // 2), (n // 2, 1), (0, 5), (7, n - 1)]
        for p in (1, 4, 5, 11):                     # both sides of strip boundaries
            cells += [(firsts[p] - 1, int(rng.integers(1, n - 1))), (firsts[p], int(rng.integers(1, n - 1)))]
        cells += [(int(i), int(j)) for i, j in rng.integers(1, n - 1, size=(6, 2))]
        fin = b0 if iters % 2 == 0 else b1
        for ci, cj in cells:
            i0, i1 = max(0, ci - iters), min(n, ci + iters + 1)
            j0, j1 = max(0, cj - iters), min(n, cj + iters + 1)
            exp = orc.jacobi_cell(grid[i0:i1, j0:j1], i0, j0, n, n, iters, ci, cj)
            p = max(q for q in range(npes) if firsts[q] <= ci)
            r = ci - firsts[p] + 1
            got = fin.gpu(p)[(r * n + cj) * 8:(r * n + cj + 1) * 8].cpu().numpy().view(np.float64)[0]
            assert np.float64(got).tobytes() == np.float64(exp).tobytes(), (ci, cj, got, exp)


def test_large_alltoall_collect_and_narrow_reduce():
    """Sizes that take the large-message launch shapes: alltoall of 8 MiB blocks and collect of
    up to 24 MiB per member on 8 PEs (whole output checked on the device), uint8 sum / xor of
    64 Mi elements through the TMA fold ring (all PEs identical + oracle windows)."""
    npes, nblk = 8, 8 * MiB
    rng = np.random.default_rng(11)
    with Session(npes, 2 * npes * nblk + 4 * MiB, with_oracle=False) as s:
        src, dst = s.malloc(npes * nblk), s.malloc(npes * nblk)
        fill_full(src, "u8", inputs.SEED_C3, npes * nblk, npes)
        B.ishmem_alltoallmem(B.ISHMEM_TEAM_WORLD, dst.addr, src.addr, nblk)
        s.sync()
        for q in range(npes):
            for i in range(npes):
                assert torch.equal(dst.gpu(q)[i * nblk:(i + 1) * nblk], src.gpu(i)[q * nblk:(q + 1) * nblk]), (q, i)
        sizes = [(3 * MiB * (i % 4)) + 4096 * i + (i % 3) for i in range(npes)]          # 0 .. ~9 MiB, ragged
        sizes[5] = 24 * MiB + 5
        assert sum(sizes) <= npes * nblk
        B.ishmem_collectmem(B.ISHMEM_TEAM_WORLD, dst.addr, src.addr, np.array(sizes, dtype=np.uint64))
        s.sync()
        at = 0
        for i in range(npes):
            for q in (0, 3, 7):
                assert torch.equal(dst.gpu(q)[at:at + sizes[i]], src.gpu(i)[:sizes[i]]), (q, i)
            at += sizes[i]
        # narrow-type reduce at a size that uses the shared-memory fold ring
        n = 64 * MiB
        o = orc.Oracle(npes, 1 << 14)
        try:
            for lop, oop in ((B.ISHMEM_OP_SUM, orc.R_SUM), (B.ISHMEM_OP_XOR, orc.R_XOR), (B.ISHMEM_OP_MAX, orc.R_MAX)):
                B.ishmemx_reduce(B.ISHMEM_TEAM_WORLD, dst.addr, src.addr, n, lop, B.ISHMEM_T_UINT8, B.ISHMEMX_REDUCE_AUTO)
                s.sync()
                for q in range(1, npes):
                    assert torch.equal(dst.gpu(q)[:n], dst.gpu(0)[:n]), (lop, q)
                for off in windows(n, 4096, rng, extra=[n // 2, n // 8 * 3]):
                    for p in range(npes):
                        o.view(0, 4096, p)[:] = inputs.block_values("u8", inputs.SEED_C3, p, off, 4096)
                    o.reduce(o.world, 8192, 0, 4096, oop, orc.T_UINT8)
                    assert np.array_equal(dst.gpu(5)[off:off + 4096].cpu().numpy(), o.view(8192, 4096, 5)), (lop, off)
        finally:
            o.close()
        assert s.status() == 0
