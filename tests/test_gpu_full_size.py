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
from tests.gpu_util import Session, heaps_equal

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


@pytest.mark.parametrize("kind,nelems", [("f32", 4 ** 13), ("f64", 4 ** 13), ("i64", 4 ** 13)])
def test_config3_reduce_large_12_pes(kind, nelems):
    """Config 3 at its largest count (4^13 = 64 Mi elements; 12 x 1 GiB of heap for the 8-byte
    types): 12 PEs, sum/max/min/prod.  Whole output: all PEs hold identical results.  Windows: the
    PE-order fold of the oracle, bit for bit (0 ulp)."""
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
    """Config 3 at its largest count: broadcast of 64 Mi float32 (256 MiB) from root 0 and
    fcollect of 64 Mi float32 per PE (3 GiB gathered on every PE, 39 GiB of heap), 12 PEs."""
    npes, nb, nf = 12, 4 * 4 ** 13, 4 * 4 ** 13
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


_GRID = {}


def config5_grid(ny, nx):
    """the seeded config-5 grid (cached: the full one is 2 GiB and three tests use it)"""
    if (ny, nx) not in _GRID:
        grid = np.empty((ny, nx))
        nblk = -(-ny // 1024)

        def gen(b):
            grid[b * 1024:min(ny, (b + 1) * 1024)] = inputs.jacobi_grid_block(inputs.SEED_C5, ny, nx, b)

        list(POOL.map(gen, range(nblk)))
        _GRID[(ny, nx)] = grid
    return _GRID[(ny, nx)]


class Strips:
    """config 5's buffers in a session: scatter a grid over the PEs' strips, run, read back"""

    def __init__(self, s, npes, ny, nx):
        self.s, self.npes, self.ny, self.nx = s, npes, ny, nx
        rows_max = -(-ny // npes)
        nbytes = (rows_max + 2) * nx * 8
        self.b0, self.b1, self.sig = s.malloc(nbytes), s.malloc(nbytes), s.malloc(64)
        base, extra = divmod(ny, npes)
        self.firsts = [p * base + min(p, extra) for p in range(npes + 1)]

    def load(self, grid):
        ny, nx = self.ny, self.nx
        for p in range(self.npes):
            lo, hi = self.firsts[p], self.firsts[p + 1]
            self.b0.gpu(p).zero_()
            self.b1.gpu(p).zero_()
            self.b0.gpu(p)[nx * 8:(hi - lo + 1) * nx * 8].copy_(torch.from_numpy(grid[lo:hi].view(np.uint8).ravel()))
            self.sig.gpu(p).zero_()
        self.s.sync()

    def run(self, iters, overlap=1):
        res = np.zeros(1)
        B.ishmemx_jacobi(self.b0.addr, self.b1.addr, self.sig.addr, self.ny, self.nx, iters, overlap, 12, 0, res)
        assert self.s.status() == 0
        self.fin = self.b0 if iters % 2 == 0 else self.b1
        return res[0]

    def strip(self, p):
        """PE p's rows of the final grid, as a device tensor of bytes"""
        lo, hi = self.firsts[p], self.firsts[p + 1]
        return self.fin.gpu(p)[self.nx * 8:(hi - lo + 1) * self.nx * 8]

    def assert_equals_grid(self, exp, what):
        for p in range(self.npes):
            lo, hi = self.firsts[p], self.firsts[p + 1]
            got = self.strip(p).cpu().numpy().view(np.uint64)
            want = exp[lo:hi].view(np.uint64).ravel()
            if not np.array_equal(got, want):
                bad = np.nonzero(got != want)[0]
                r, c = divmod(int(bad[0]), self.nx)
                raise AssertionError(f"{what}: PE {p} differs from the oracle in {bad.size} cells, first at "
                                     f"global row {lo + r}, column {c}")

    def cell(self, ci, cj):
        p = max(q for q in range(self.npes) if self.firsts[q] <= ci)
        r = ci - self.firsts[p] + 1
        return self.fin.gpu(p)[(r * self.nx + cj) * 8:(r * self.nx + cj + 1) * 8].cpu().numpy().view(np.float64)[0]


def test_config5_jacobi_16384_whole_grid_even_and_odd_sweep_counts():
    """Config 5 at full size in the launch shape the library picks by itself, 12 PEs: the WHOLE
    final grid bit for bit against the oracle's plain full-grid sweeps, and the residual at 1e-6
    relative, for 8 sweeps (two launches of four), 9 (three launches of three), 12 (two launches of
    six) and 17 (six, six and five) -- every band and tile-group seam and all eleven strip seams are
    compared.  The later oracle grids continue from the earlier ones (a sweep has no memory, which
    a CPU test pins)."""
    npes, n = 12, 16384
    grid = config5_grid(n, n)
    u8, r8 = orc.jacobi(grid, 8)
    u9, r9 = orc.jacobi(u8, 1)
    u12, r12 = orc.jacobi(u9, 3)
    u17, r17 = orc.jacobi(u12, 5)
    out = np.zeros(8, dtype=np.int32)
    assert B.ishmemx_jacobi_launch_depths(12, 6, out, 8) == 2 and out[:2].tolist() == [6, 6]
    assert B.ishmemx_jacobi_launch_depths(17, 6, out, 8) == 3 and out[:3].tolist() == [6, 6, 5]
    rows_max = -(-n // npes)
    with Session(npes, 2 * (rows_max + 2) * n * 8 + 2 * MiB, with_oracle=False) as s:
        st = Strips(s, npes, n, n)
        for iters, exp, exp_res in ((8, u8, r8), (9, u9, r9), (12, u12, r12), (17, u17, r17)):
            st.load(grid)
            res = st.run(iters)
            st.assert_equals_grid(exp, f"{iters} sweeps")
            assert abs(res - exp_res) <= 1e-6 * exp_res, (iters, res, exp_res)


def test_config5_jacobi_full_width_200_sweeps_whole_grid_and_residual():
    """200 sweeps on rows of config 5's full width (16384 columns x 768 rows, 12 strips of one
    64-row band each): whole grid and residual against the oracle, in the form that the library uses
    at full size (four columns per lane, up to six sweeps per launch), on a grid small enough for any
    host."""
    npes, ny, nx, iters = 12, 768, 16384, 200
    grid = config5_grid(ny, nx)
    exp, exp_res = orc.jacobi(grid, iters)
    with Session(npes, 2 * (ny // npes + 2) * nx * 8 + 2 * MiB, with_oracle=False) as s:
        B.ishmemx_set_option(B.ISHMEMX_OPT_JACOBI_WIDE, 1)
        st = Strips(s, npes, ny, nx)
        st.load(grid)
        res = st.run(iters)
        st.assert_equals_grid(exp, "200 sweeps, full-width rows")
        assert abs(res - exp_res) <= 1e-6 * exp_res, (res, exp_res)


def test_config5_jacobi_16384_200_iterations_sampled_cells():
    """Config 5 at full size: 16384 x 16384 float64, 12 row strips, 200 sweeps with in-kernel
    put_signal halos.  Sampled cells -- corners, edges, both sides of strip boundaries, of band
    seams (every 16, 64 and 128 rows of a strip) and of tile seams (every 56, 60, 112, 120, 448 and
    960 columns), interior -- are compared bit for bit with the oracle's dependency-cone evaluation
    from the initial grid; then the whole final grid and the L2 residual with the oracle's 200
    full-grid sweeps.  Last, the same 200 sweeps as single-sweep launches: every strip and the
    residual must agree with the default form's."""
    npes, n, iters = 12, 16384, 200
    grid = config5_grid(n, n)
    rows_max = -(-n // npes)
    with Session(npes, 2 * (rows_max + 2) * n * 8 + 2 * MiB, with_oracle=False) as s:
        st = Strips(s, npes, n, n)
        firsts = st.firsts
        st.load(grid)
        res = st.run(iters)
        rng = np.random.default_rng(10)
        cells = [(1, 1), (n - 2, n - 2), (1, n // 2), (n // 2, 1), (0, 5), (7, n - 1)]
        for p in (1, 4, 5, 11):                     # both sides of strip boundaries
            cells += [(firsts[p] - 1, int(rng.integers(1, n - 1))), (firsts[p], int(rng.integers(1, n - 1)))]
        for band, tile in ((64, 120), (64, 960), (16, 60), (64, 56), (16, 480), (64, 448), (128, 112), (128, 448)):
            p, k, t = int(rng.integers(0, npes)), int(rng.integers(1, 1300 // band)), int(rng.integers(1, n // tile))
            row = firsts[p] + band * k              # first row of band k of strip p
            cells += [(row - 1, tile * t - 1), (row, tile * t), (row - 1, tile * t), (row, tile * t - 1)]
        cells += [(int(i), int(j)) for i, j in rng.integers(1, n - 1, size=(6, 2))]

        def check(cell):
            ci, cj = cell
            i0, i1 = max(0, ci - iters), min(n, ci + iters + 1)
            j0, j1 = max(0, cj - iters), min(n, cj + iters + 1)
            return orc.jacobi_cell(grid[i0:i1, j0:j1], i0, j0, n, n, iters, ci, cj)

        for (ci, cj), exp in zip(cells, POOL.map(check, cells)):
            got = st.cell(ci, cj)
            assert np.float64(got).tobytes() == np.float64(exp).tobytes(), (ci, cj, got, exp)
        # the oracle's 200 plain full-grid sweeps (5.4 x 10^10 cell updates on one host core: about
        # a minute on a server CPU): the whole final grid bit for bit, the residual at 1e-6
        exp, exp_res = orc.jacobi(grid, iters)
        st.assert_equals_grid(exp, "200 sweeps")
        assert abs(res - exp_res) <= 1e-6 * exp_res, (res, exp_res)
        del exp
        # the same run as 200 single-sweep launches
        fused = [st.strip(p).clone() for p in range(npes)]      # 2 GiB of torch memory beside the heap
        B.ishmemx_set_option(B.ISHMEMX_OPT_JACOBI_FUSE, 0)
        st.load(grid)
        res1 = st.run(iters)
        for p in range(npes):
            assert torch.equal(st.strip(p), fused[p]), p
        assert abs(res - res1) <= 1e-6 * res1, (res, res1)


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


@pytest.mark.parametrize("level,n,threads", [(B.ISHMEMX_WORK_ITEM, 4 * MiB, 1), (B.ISHMEMX_SUB_GROUP, 64 * MiB, 32)])
def test_config2_one_thread_and_one_warp_at_their_largest_sweep_sizes(level, n, threads):
    """The largest messages the size sweep times for a single work-item (4 MiB) and a single
    sub-group (64 MiB): ONE collaboration unit moves the whole message, put and get, with
    unaligned ends; every byte of both heaps against the oracle."""
    npes = 2
    with Session(npes, 2 * n + MiB) as s:
        src, dst = s.malloc(n), s.malloc(n)
        for p in range(npes):
            src.fill(p, inputs.byte_payload(inputs.SEED_C2, 40 + p, n))
        m = n - 3                                        # ragged tail; head at offset 1: misaligned by one
        B.ishmemx_putmem_on_device(0, dst.addr + 1, src.addr + 1, m - 1, 1, level, threads, 1)
        s.oracle.putmem(0, dst.ooff + 1, s.oracle.ptr(src.ooff + 1, m - 1, 0), m - 1, 1)
        B.ishmemx_getmem_on_device(0, dst.addr, src.addr, n, 1, level, threads, 1)       # PE 0 <- PE 1's src
        s.oracle.getmem(0, s.oracle.ptr(dst.ooff, n, 0), src.ooff, n, 1)
        B.ishmem_barrier_all()
        heaps_equal(s, f"level {level}, {n} bytes")
        assert s.status() == 0
