"""Pins for the oracle's Jacobi overlap workload: a hand-computed case, the
discrete sine eigenmode's closed-form decay, the maximum principle, and
independence of the result from the strip decomposition and from the
dependency-cone shortcut."""
from pathlib import Path

import numpy as np
import pytest

import oracle as orc
from oracle import Oracle
from paper_2409_20476_b200 import inputs

GOLD = Path(__file__).parent / "golden" / "jacobi_4x4_hand.txt"


def read_gold():
    out = {}
    for line in GOLD.read_text().splitlines():
        if not line or line.startswith("#"):
            continue
        k, *v = line.split()
        out[k] = np.array([float(x) for x in v])
    return out


def test_hand_computed_4x4():
    g = read_gold()
    u1, _ = orc.jacobi(g["init"].reshape(4, 4), 1)
    assert np.array_equal(u1.ravel(), g["sweep1"])
    u2, r2 = orc.jacobi(g["init"].reshape(4, 4), 2)
    assert np.array_equal(u2.ravel(), g["sweep2"])
    assert r2 == g["residual_sq2"][0]


def test_zero_grid_stays_zero_and_zero_iters_is_identity():
    u, r = orc.jacobi(np.zeros((9, 7)), 5)
    assert not u.any() and r == 0.0
    g = inputs.jacobi_grid(4, 6, 5)
    u, _ = orc.jacobi(g, 0)
    assert np.array_equal(u, g)


def test_asymmetric_stencil_orientation():
    """A single 1 spreads to exactly its four neighbours with weight 1/4 (catches a
    transposed index or a dropped neighbour)."""
    g = np.zeros((7, 9))
    g[2, 5] = 1.0
    u, _ = orc.jacobi(g, 1)
    exp = np.zeros((7, 9))
    for di, dj in ((-1, 0), (1, 0), (0, -1), (0, 1)):
        exp[2 + di, 5 + dj] = 0.25
    assert np.array_equal(u, exp)
    # next to the boundary the ring stays 0
    g = np.zeros((5, 5))
    g[1, 1] = 1.0
    u, _ = orc.jacobi(g, 1)
    assert u[0, 1] == 0 and u[1, 0] == 0 and u[1, 2] == 0.25 and u[2, 1] == 0.25


@pytest.mark.parametrize("ny,nx", [(10, 10), (8, 13)])
def test_eigenmode_decay(ny, nx):
    """sin(pi i/(ny-1)) sin(pi j/(nx-1)) is an eigenvector of the sweep with eigenvalue
    0.5*(cos(pi/(ny-1)) + cos(pi/(nx-1)))."""
    i = np.arange(ny)[:, None]
    j = np.arange(nx)[None, :]
    mode = np.sin(np.pi * i / (ny - 1)) * np.sin(np.pi * j / (nx - 1))
    mode[0, :] = mode[-1, :] = 0.0
    mode[:, 0] = mode[:, -1] = 0.0
    lam = 0.5 * (np.cos(np.pi / (ny - 1)) + np.cos(np.pi / (nx - 1)))
    k = 25
    u, r = orc.jacobi(mode, k)
    assert np.allclose(u, lam**k * mode, rtol=1e-12, atol=1e-15)
    # last update = (lam^k - lam^(k-1)) * mode
    exp_r = ((lam**k - lam**(k - 1)) ** 2) * (mode[1:-1, 1:-1] ** 2).sum()
    assert abs(r - exp_r) <= 1e-10 * exp_r


def test_maximum_principle():
    g = inputs.jacobi_grid(4, 40, 33)
    prev = g.max()
    for k in (1, 2, 5, 20):
        u, _ = orc.jacobi(g, k)
        assert u.min() >= 0.0 and u.max() <= prev + 1e-18
        prev = u.max()


def run_strips(grid, npes, iters):
    ny, nx = grid.shape
    rows_max = -(-ny // npes)
    nbytes = (rows_max + 2) * nx * 8
    o = Oracle(npes, 2 * nbytes + 4096)
    b0 = o.malloc(nbytes)
    b1 = o.malloc(nbytes)
    sig = o.malloc(16)
    o.jacobi_scatter(b0, grid)
    res = o.jacobi_strips(b0, b1, sig, ny, nx, iters)
    final = o.jacobi_gather(b0 if iters % 2 == 0 else b1, ny, nx)
    return final, res


@pytest.mark.parametrize("npes", [1, 2, 5, 12])
@pytest.mark.parametrize("iters", [1, 2, 7])
def test_strip_decomposition_independent(npes, iters):
    """The PE program with put_signal halo exchange gives the full-grid result bit for bit."""
    g = inputs.jacobi_grid(4, 29, 17)
    full, rfull = orc.jacobi(g, iters)
    strips, rstrips = run_strips(g, npes, iters)
    assert strips.tobytes() == full.tobytes()
    assert abs(rstrips - rfull) <= 1e-12 * rfull


def test_strip_rows_partition():
    o = Oracle(12, 64)
    firsts, rows = zip(*[o.jacobi_strip_rows(16384, p) for p in range(12)])
    assert rows == (1366,) * 4 + (1365,) * 8          # 16384 = 12*1365 + 4
    assert firsts[0] == 0 and all(firsts[p + 1] == firsts[p] + rows[p] for p in range(11))
    assert firsts[-1] + rows[-1] == 16384


@pytest.mark.parametrize("ci,cj", [(20, 20), (0, 7), (3, 1), (39, 30), (12, 31), (38, 1)])
def test_cell_cone_equals_full_grid(ci, cj):
    ny, nx, iters = 40, 32, 6
    g = inputs.jacobi_grid(4, ny, nx)
    full, _ = orc.jacobi(g, iters)
    i0, i1 = max(0, ci - iters), min(ny, ci + iters + 1)
    j0, j1 = max(0, cj - iters), min(nx, cj + iters + 1)
    v = orc.jacobi_cell(g[i0:i1, j0:j1], i0, j0, ny, nx, iters, ci, cj)
    assert v == full[ci, cj]
    if i0 > 0:  # a window that does not hold the cone is refused
        with pytest.raises(orc.OracleError):
            orc.jacobi_cell(g[i0 + 1:i1, j0:j1], i0 + 1, j0, ny, nx, iters, ci, cj)


def test_blocked_grid_generator_windows():
    ny, nx = 2500, 40
    blocks = [inputs.jacobi_grid_block(4, ny, nx, b) for b in range(3)]
    full = np.concatenate(blocks)
    assert full.shape == (ny, nx)
    assert not full[0].any() and not full[-1].any() and not full[:, 0].any()
    win = inputs.jacobi_cell_init(4, ny, nx, 1000, 1100, 3, 30)
    assert np.array_equal(win, full[1000:1100, 3:30])


GOLD_ASSOC = Path(__file__).parent / "golden" / "jacobi_3x3_association.txt"


def read_gold_assoc():
    out = {}
    for line in GOLD_ASSOC.read_text().splitlines():
        if not line or line.startswith("#"):
            continue
        k, *v = line.split()
        out[k] = np.array([float(x) for x in v])
    return out


def test_association_order_of_the_update_is_pinned():
    """(N+S)+(W+E), fixed by a case in which every other order of the three additions gives
    a different float64 (0.0 against 0.25 or 0.5): full grid, PE program and cone form."""
    g = read_gold_assoc()
    init = g["init"].reshape(3, 3)
    # the hand derivation's premises hold in this arithmetic
    assert np.float64(1e16) + np.float64(1.0) == np.float64(1e16)
    assert g["wrong_left_to_right"][0] == 0.25 * (((init[0, 1] + init[2, 1]) + init[1, 0]) + init[1, 2])
    assert g["wrong_pair_by_axis_swapped"][0] == 0.25 * ((init[0, 1] + init[1, 0]) + (init[2, 1] + init[1, 2]))
    u, r = orc.jacobi(init, 1)
    assert u.tobytes() == g["sweep1"].reshape(3, 3).tobytes()
    assert r == g["residual_sq1"][0]
    for npes in (1, 3):   # 3 PEs: one row each, N and S arrive through the put_signal halos
        strips, rs = run_strips(init, npes, 1)
        assert strips.tobytes() == g["sweep1"].reshape(3, 3).tobytes()
        assert rs == g["residual_sq1"][0]
    assert orc.jacobi_cell(init, 0, 0, 3, 3, 1, 1, 1) == 0.0
    # the same stencil embedded in a larger grid, so that the cone form takes its interior
    # branch with a window that is not the whole grid
    big = np.zeros((7, 8))
    big[2:5, 3:6] = init
    full, _ = orc.jacobi(big, 1)
    assert full[3, 4] == 0.0
    assert orc.jacobi_cell(big[2:5, 3:6], 2, 3, 7, 8, 1, 3, 4) == 0.0


def test_sweeps_compose():
    """k sweeps followed by m sweeps of the result are k + m sweeps, bit for bit, and the
    residual is that of the last sweep alone (the full-size GPU test continues the oracle's
    eighth sweep into a ninth)."""
    g = inputs.jacobi_grid(4, 37, 22)
    u8, _ = orc.jacobi(g, 8)
    u9, r9 = orc.jacobi(g, 9)
    v9, s9 = orc.jacobi(u8, 1)
    assert v9.tobytes() == u9.tobytes() and s9 == r9
    w9, t9 = orc.jacobi(orc.jacobi(g, 4)[0], 5)
    assert w9.tobytes() == u9.tobytes() and t9 == r9
