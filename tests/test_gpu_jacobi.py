"""GPU parity of the overlap workload (config 5): in-kernel put_signal halo exchange around
a 5-point Jacobi sweep, final grid bit-exact against the CPU oracle, residual at 1e-6."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2409_20476_b200 import binding as B
from paper_2409_20476_b200 import inputs
from tests.gpu_util import Session

pytestmark = pytest.mark.gpu


def run_gpu(grid, npes, iters, overlap, groups, threads, options=(), spare_rows=8, want_residual=True):
    """spare_rows: rows of symmetric heap left free beside the two buffers -- launches of three to six
    sweeps park their deeper halo rows in up to eight rows that the library allocates for the call"""
    ny, nx = grid.shape
    rows_max = -(-ny // npes)
    nbytes = (rows_max + 2) * nx * 8
    with Session(npes, 2 * nbytes + (1 << 12) + spare_rows * nx * 8, with_oracle=False) as s:
        for opt, value in options:
            B.ishmemx_set_option(opt, value)
        b0, b1, sig = s.malloc(nbytes), s.malloc(nbytes), s.malloc(64)
        base, extra = divmod(ny, npes)
        first = 0
        for p in range(npes):
            rows = base + (1 if p < extra else 0)
            strip = np.zeros((rows_max + 2, nx))
            strip[1:rows + 1] = grid[first:first + rows]
            b0.fill(p, strip)
            sig.fill(p, np.zeros(64, np.uint8))
            first += rows
        res = np.zeros(1)
        B.ishmemx_jacobi(b0.addr, b1.addr, sig.addr, ny, nx, iters, overlap, groups, threads,
                         res if want_residual else None)
        assert s.status() == 0
        out = np.zeros_like(grid)
        fin = b0 if iters % 2 == 0 else b1
        first = 0
        for p in range(npes):
            rows = base + (1 if p < extra else 0)
            out[first:first + rows] = fin.read(p, np.float64).reshape(rows_max + 2, nx)[1:rows + 1]
            first += rows
        return out, res[0]


SWEEP_FORMS = {   # (sweeps per launch at most: 1 = the library's choice, up to six; four columns per lane)
    "sweeps": (1, 1), "sweeps_two_columns_per_lane": (1, 0), "two_per_launch": (2, 1),
    "three_per_launch_two_columns_per_lane": (3, 0), "four_per_launch": (4, 1),
    "five_per_launch_two_columns_per_lane": (5, 0), "five_per_launch": (5, 1), "single_sweeps": (0, 1)}


@pytest.mark.parametrize("split", list(SWEEP_FORMS) + ["columns", "rows"])
@pytest.mark.parametrize("overlap", [1, 0])
@pytest.mark.parametrize("ny,nx,npes,groups,threads", [
    (64, 48, 12, 1, 128), (200, 131, 12, 3, 128), (257, 33, 5, 4, 128),       # odd nx: row-by-row path
    (40, 40, 1, 2, 128), (1000, 512, 12, 8, 128), (301, 1234, 7, 3, 256),      # sliding window, 128 registers
    (600, 256, 12, 13, 128), (300, 4096, 4, 2, 1024), (97, 62, 3, 5, 1024),    # sliding window, 64 registers
    (120, 2880, 6, 6, 0), (90, 1442, 3, 2, 0), (60, 5000, 2, 4, 640),          # threads chosen by the library; 80 registers
    (36, 600, 12, 12, 32), (50, 121, 4, 3, 64)])                               # one tile per block; odd nx by columns
def test_jacobi_matches_oracle(ny, nx, npes, groups, threads, overlap, split):
    """split: the persistent kernel with the strips cut by columns or by rows, or one of the launch-ordered
    forms that the library uses for threads = 0 and even nx: `sweeps` = its own choice (one tile per warp, up
    to six sweeps per launch, four columns per lane where nx is a multiple of 4), the same with two columns
    per lane, with at most two to five sweeps per launch, or with one sweep per launch.  The 21 sweeps are
    cut into launches by ishmemx_jacobi_launch_depths (an odd number of them, deepest first)."""
    if split in SWEEP_FORMS:
        options = [(B.ISHMEMX_OPT_JACOBI_SPLIT, 0), (B.ISHMEMX_OPT_JACOBI_FUSE, SWEEP_FORMS[split][0]),
                   (B.ISHMEMX_OPT_JACOBI_WIDE, SWEEP_FORMS[split][1])]
        threads = 0
    else:
        options = [(B.ISHMEMX_OPT_JACOBI_SPLIT, {"rows": 1, "columns": 2}[split])]
    grid = inputs.jacobi_grid(inputs.SEED_C5, ny, nx)
    iters = 21
    exp, exp_res = orc.jacobi(grid, iters)
    got, res = run_gpu(grid, npes, iters, overlap, groups, threads, options)
    assert got.tobytes() == exp.tobytes()
    assert abs(res - exp_res) <= 1e-6 * exp_res


def test_jacobi_default_split_and_repeated_calls():
    """With the options at their defaults: threads = 0 launches once per sweep, a given block size runs the persistent
    kernel with the strips cut by rows; both give the oracle's grid."""
    grid = inputs.jacobi_grid(inputs.SEED_C5, 150, 2400)         # 40 column tiles
    exp, _ = orc.jacobi(grid, 9)
    for groups, threads in ((2, 0), (5, 0), (5, 96), (40, 0)):    # one launch per sweep; (5, 96): persistent, by rows
        got, _ = run_gpu(grid, 6, 9, 1, groups, threads)
        assert got.tobytes() == exp.tobytes(), (groups, threads)


def test_jacobi_per_sweep_many_bands_and_residual():
    """The launch-ordered form on strips of several bands and tile groups, with strips of unequal length and
    iteration counts whose last launch -- the one that forms the residual -- is one of 1 to 6 sweeps, with
    room in the heap for all the deeper halo rows (8), for those of four sweeps per launch (4) and for none
    (launches then stay at two sweeps); final grid bit-exact, residual within 1e-6 relative."""
    grid = inputs.jacobi_grid(inputs.SEED_C5, 1000, 1100)
    for npes, iters, spare in ((7, 5, 8), (3, 12, 8), (1, 3, 8), (5, 8, 8), (12, 4, 8), (2, 10, 8), (6, 6, 8),
                               (7, 8, 0), (3, 5, 0), (4, 22, 8), (4, 16, 0), (4, 22, 4), (3, 12, 4), (5, 18, 8),
                               (2, 11, 8), (1, 6, 8), (3, 24, 5)):
        exp, exp_res = orc.jacobi(grid, iters)
        got, res = run_gpu(grid, npes, iters, 1, 1, 0, spare_rows=spare)
        assert got.tobytes() == exp.tobytes(), (npes, iters, spare)
        assert abs(res - exp_res) <= 1e-6 * exp_res


def test_jacobi_multi_sweep_launches_on_the_shortest_strips():
    """Strips of one to seven rows: a launch is at most as deep as the shortest strip has rows (it sends that many
    of its rows each way), the deeper halo rows of a neighbour are its rows next to the edge row, and a strip's
    single band is both its first and its last."""
    for ny, nx, npes in ((24, 120, 12), (31, 232, 10), (8, 64, 4), (12, 128, 12), (48, 240, 12), (50, 484, 10),
                         (72, 120, 12), (26, 232, 4), (6, 64, 1)):
        grid = inputs.jacobi_grid(inputs.SEED_C5, ny, nx)
        for iters in (4, 8, 9, 12):
            exp, exp_res = orc.jacobi(grid, iters)
            got, res = run_gpu(grid, npes, iters, 1, 1, 0)
            assert got.tobytes() == exp.tobytes(), (ny, nx, npes, iters)
            assert abs(res - exp_res) <= 1e-6 * exp_res


def test_jacobi_launch_ordered_forms_on_random_shapes():
    """Seeded random shapes for the launch-ordered form: grids from a few cells to several bands and tile groups
    (one, two and more tile groups per band; strips shorter than a launch is deep; strips of unequal length;
    widths with and without a multiple of four), any cap on the sweeps per launch, both column widths, with and
    without overlap, with and without a residual, with room in the heap for all, some or none of the deeper halo
    rows.  Grid bit-exact, residual within 1e-6 relative."""
    rng = np.random.default_rng(20240917)
    for case in range(60):
        npes = int(rng.integers(1, 13))
        ny = int(rng.integers(max(3, npes), 700))
        nx = 2 * int(rng.integers(2, 1100 if case % 3 else 160))
        iters = int(rng.integers(1, 20))
        fuse, wide = int(rng.integers(0, 7)), int(rng.integers(-1, 2))
        overlap, want, spare = int(rng.integers(0, 2)), bool(rng.integers(0, 2)), int(rng.choice([0, 2, 4, 6, 8]))
        grid = inputs.jacobi_grid(inputs.SEED_C5 + case, ny, nx)
        exp, exp_res = orc.jacobi(grid, iters)
        options = [(B.ISHMEMX_OPT_JACOBI_FUSE, fuse), (B.ISHMEMX_OPT_JACOBI_WIDE, wide)]
        got, res = run_gpu(grid, npes, iters, overlap, 1, 0, options, spare_rows=spare, want_residual=want)
        what = (case, npes, ny, nx, iters, fuse, wide, overlap, want, spare)
        assert got.tobytes() == exp.tobytes(), what
        if want:
            assert abs(res - exp_res) <= 1e-6 * exp_res + 1e-300, what


def test_jacobi_without_residual():
    """residual_sq_host = NULL: the last launch forms no residual (in the launch-ordered form it then runs
    like the others); the grid is the oracle's all the same."""
    grid = inputs.jacobi_grid(inputs.SEED_C5, 700, 1200)
    for npes, iters, threads in ((5, 12, 0), (3, 7, 0), (1, 6, 0), (4, 9, 128)):
        exp, _ = orc.jacobi(grid, iters)
        got, res = run_gpu(grid, npes, iters, 1, 2, threads, want_residual=False)
        assert got.tobytes() == exp.tobytes(), (npes, iters, threads)
        assert res == 0.0


def test_jacobi_even_iterations_and_zero():
    grid = inputs.jacobi_grid(inputs.SEED_C5, 96, 64)
    for iters in (0, 1, 2, 10):
        exp, _ = orc.jacobi(grid, iters)
        got, _ = run_gpu(grid, 12, iters, 1, 2, 64)
        assert got.tobytes() == exp.tobytes(), iters


def test_refused_coresident_launch_leaves_the_library_usable():
    """A persistent launch that cannot be co-resident is refused with NOT_CORESIDENT; the
    refusal must not leak into the next call."""
    npes, ny, nx = 12, 4800, 60 * 400        # 400 rows and 400 column tiles per strip: no clamping of the groups
    nbytes = (ny // npes + 2) * nx * 8
    with Session(npes, 2 * nbytes + (1 << 16), with_oracle=False) as s:
        b0, b1, sig = s.malloc(nbytes), s.malloc(nbytes), s.malloc(64)
        with pytest.raises(B.IshmemError) as e:
            B.ishmemx_jacobi(b0.addr, b1.addr, sig.addr, ny, nx, 2, 1, 400, 1024, None)
        assert e.value.code == B.ISHMEM_ERR_NOT_CORESIDENT
        B.ishmem_uint64_p(0, sig.addr, 5, 1)
        B.ishmem_barrier_all()
        assert sig.read(1, np.uint64)[0] == 5
        assert s.status() == 0
