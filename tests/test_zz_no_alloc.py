"""The allocation-free Jacobi entry point against the regular one and against the CPU oracle.

``ishmemx_jacobi_noalloc`` exists for callers that cannot allocate device memory when they
call the library (a frozen memory pool, a loop that must not hit cudaMalloc's device-wide
synchronisation, an allocator that owns the whole GPU): its kernel scratch lives in a fixed
device array inside the library instead of a fresh allocation.  It must give exactly what
``ishmemx_jacobi`` gives and what the oracle's plain full-grid sweeps give -- the same final
grid bit for bit, the residual within 1e-6 relative -- and, because the shared array keeps the
previous call's contents, it must do so on two calls in a row.  The second call must also
leave the device's free memory exactly where it found it (the first call of a process may
load the kernel's code).  This file sorts last so that a run stopping at the first failure
has already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2409_20476_b200 import binding as B
from paper_2409_20476_b200 import inputs
from tests.gpu_util import Session

pytestmark = pytest.mark.gpu


def load_strips(s, buf, grid, npes, rows_max):
    ny, nx = grid.shape
    base, extra = divmod(ny, npes)
    first = 0
    for p in range(npes):
        rows = base + (1 if p < extra else 0)
        strip = np.zeros((rows_max + 2, nx))
        strip[1:rows + 1] = grid[first:first + rows]
        buf.fill(p, strip)
        first += rows


def run(fn, s, b0, b1, sig, grid, npes, rows_max, iters, groups, threads):
    load_strips(s, b0, grid, npes, rows_max)
    for p in range(npes):
        b1.fill(p, np.zeros(b1.nbytes, np.uint8))
        sig.fill(p, np.zeros(64, np.uint8))
    res = np.zeros(1)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    fn(b0.addr, b1.addr, sig.addr, grid.shape[0], grid.shape[1], iters, 1, groups, threads, res)
    free_after = torch.cuda.mem_get_info()[0]
    assert s.status() == 0
    fin = b0 if iters % 2 == 0 else b1
    return [fin.read(p).copy() for p in range(npes)], res[0], free_before - free_after


def assert_is_oracle_grid(strips, res, grid, iters, npes):
    """the strips (one halo row above and below each) against the oracle's full-grid sweeps"""
    exp, exp_res = orc.jacobi(grid, iters)
    ny, nx = grid.shape
    base, extra = divmod(ny, npes)
    first = 0
    for p in range(npes):
        rows = base + (1 if p < extra else 0)
        got = strips[p].view(np.float64).reshape(-1, nx)[1:rows + 1]
        assert got.tobytes() == exp[first:first + rows].tobytes(), f"PE {p} differs from the oracle"
        first += rows
    assert abs(res - exp_res) <= 1e-6 * exp_res


def test_noalloc_matches_regular_entry_point_twice():
    npes, ny, nx, groups, threads = 12, 300, 96, 4, 128
    rows_max = -(-ny // npes)
    nbytes = (rows_max + 2) * nx * 8
    grid = inputs.jacobi_grid(inputs.SEED_C5, ny, nx)
    with Session(npes, 2 * nbytes + (1 << 16), with_oracle=False) as s:
        b0, b1, sig = s.malloc(nbytes), s.malloc(nbytes), s.malloc(64)
        ref, ref_res, _ = run(B.ishmemx_jacobi, s, b0, b1, sig, grid, npes, rows_max, 13, groups, threads)
        assert_is_oracle_grid(ref, ref_res, grid, 13, npes)
        for call in range(2):   # second call finds the first call's counters in the shared array
            got, res, used = run(B.ishmemx_jacobi_noalloc, s, b0, b1, sig, grid, npes, rows_max, 13, groups, threads)
            assert_is_oracle_grid(got, res, grid, 13, npes)
            for p in range(npes):
                assert got[p].tobytes() == ref[p].tobytes(), (call, p)
            assert abs(res - ref_res) <= 1e-6 * ref_res
            if call == 1:       # nothing was allocated on the device, not even transiently kept
                assert used == 0, f"free device memory changed by {used} bytes across the call"
        # a different shape right after (fewer blocks, fewer sweeps) still starts from clean counters
        ref2, ref2_res, _ = run(B.ishmemx_jacobi, s, b0, b1, sig, grid, npes, rows_max, 4, 2, 64)
        got2, res2, used2 = run(B.ishmemx_jacobi_noalloc, s, b0, b1, sig, grid, npes, rows_max, 4, 2, 64)
        assert_is_oracle_grid(got2, res2, grid, 4, npes)
        for p in range(npes):
            assert got2[p].tobytes() == ref2[p].tobytes()
        assert abs(res2 - ref2_res) <= 1e-6 * ref2_res
        assert used2 == 0


def test_noalloc_rejects_launches_beyond_its_fixed_scratch():
    npes, ny, nx = 12, 12 * 200, 60 * 171    # enough rows and column tiles that 171 groups are not clamped
    rows_max = ny // npes
    nbytes = (rows_max + 2) * nx * 8
    with Session(npes, 2 * nbytes + (1 << 16), with_oracle=False) as s:
        b0, b1, sig = s.malloc(nbytes), s.malloc(nbytes), s.malloc(64)
        with pytest.raises(B.IshmemError) as e:      # 12 x 171 = 2052 blocks > 2048
            B.ishmemx_jacobi_noalloc(b0.addr, b1.addr, sig.addr, ny, nx, 1, 1, 171, 32, None)
        assert e.value.code == B.ISHMEM_ERR_ARG
        assert "2048" in B.ishmemx_last_cuda_error().decode()
        assert s.status() == 0
