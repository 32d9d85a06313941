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


def run_gpu(grid, npes, iters, overlap, groups, threads, options=()):
    ny, nx = grid.shape
    rows_max = -(-ny // npes)
    nbytes = (rows_max + 2) * nx * 8
    with Session(npes, 2 * nbytes + (1 << 16), with_oracle=False) as s:
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
        B.ishmemx_jacobi(b0.addr, b1.addr, sig.addr, ny, nx, iters, overlap, groups, threads, res)
        assert s.status() == 0
        out = np.zeros_like(grid)
        fin = b0 if iters % 2 == 0 else b1
        first = 0
        for p in range(npes):
            rows = base + (1 if p < extra else 0)
            out[first:first + rows] = fin.read(p, np.float64).reshape(rows_max + 2, nx)[1:rows + 1]
            first += rows
        return out, res[0]


@pytest.mark.parametrize("split", ["sweeps", "sweeps_two_columns_per_lane", "single_sweeps", "columns", "rows"])
@pytest.mark.parametrize("overlap", [1, 0])
@pytest.mark.parametrize("ny,nx,npes,groups,threads", [
    (64, 48, 12, 1, 128), (200, 131, 12, 3, 128), (257, 33, 5, 4, 128),       # odd nx: row-by-row path
    (40, 40, 1, 2, 128), (1000, 512, 12, 8, 128), (301, 1234, 7, 3, 256),      # sliding window, 128 registers
    (600, 256, 12, 13, 128), (300, 4096, 4, 2, 1024), (97, 62, 3, 5, 1024),    # sliding window, 64 registers
    (120, 2880, 6, 6, 0), (90, 1442, 3, 2, 0), (60, 5000, 2, 4, 640),          # threads chosen by the library; 80 registers
    (36, 600, 12, 12, 32), (50, 121, 4, 3, 64)])                               # one tile per block; odd nx by columns
def test_jacobi_matches_oracle(ny, nx, npes, groups, threads, overlap, split):
    """split: the persistent kernel with the strips cut by columns or by rows, or `sweeps`: the form the
    library picks by itself for threads = 0 and even nx (one tile per warp, two sweeps per launch where the
    count allows, four columns per lane), the same with two columns per lane, or with one sweep per launch."""
    if split in ("sweeps", "sweeps_two_columns_per_lane", "single_sweeps"):
        options = [(B.ISHMEMX_OPT_JACOBI_SPLIT, 0),
                   (B.ISHMEMX_OPT_JACOBI_FUSE, 0 if split == "single_sweeps" else 1),
                   (B.ISHMEMX_OPT_JACOBI_WIDE, 0 if split == "sweeps_two_columns_per_lane" else 1)]
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
    """The launch-per-sweep form on strips of several bands and tile groups, with strips of unequal length and
    iteration counts that end in a two-sweep pass or in one to three single sweeps; final grid bit-exact,
    residual within 1e-6 relative."""
    grid = inputs.jacobi_grid(inputs.SEED_C5, 1000, 1100)
    for npes, iters in ((7, 5), (3, 12), (1, 3), (5, 8), (12, 4), (2, 10)):     # 2, 6, 0, 4, 2, 4 two-sweep passes
        exp, exp_res = orc.jacobi(grid, iters)
        got, res = run_gpu(grid, npes, iters, 1, 1, 0)
        assert got.tobytes() == exp.tobytes(), (npes, iters)
        assert abs(res - exp_res) <= 1e-6 * exp_res


def test_jacobi_two_sweep_passes_on_the_shortest_strips():
    """Strips of two and three rows: the second halo row of a neighbour is its first or last row but one, and a
    strip's single band is both its first and its last; 4 and 8 sweeps are all two-sweep passes."""
    for ny, nx, npes in ((24, 120, 12), (31, 232, 10), (8, 64, 4)):
        grid = inputs.jacobi_grid(inputs.SEED_C5, ny, nx)
        for iters in (4, 8, 9):
            exp, exp_res = orc.jacobi(grid, iters)
            got, res = run_gpu(grid, npes, iters, 1, 1, 0)
            assert got.tobytes() == exp.tobytes(), (ny, nx, npes, iters)
            assert abs(res - exp_res) <= 1e-6 * exp_res


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
