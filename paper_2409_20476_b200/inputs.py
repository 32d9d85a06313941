"""Seeded synthetic workloads, shared by the tests and the benchmark.

This module only draws random inputs with the shapes and value distributions of
the five benchmark configurations; it contains none of the library's
arithmetic and imports neither the CUDA binding nor the CPU oracle.  The same
arrays are handed to both sides.
"""
from __future__ import annotations

import numpy as np

SEED_C1, SEED_C2, SEED_C3, SEED_C4, SEED_C5 = 0, 1, 2, 3, 4


def rng_for(seed: int, *stream) -> np.random.Generator:
    """Independent generator per (seed, stream...) so that sizes do not shift each other."""
    return np.random.default_rng([seed, *[int(s) for s in stream]])


def int32_payload(seed: int, pe: int, nelems: int) -> np.ndarray:
    """Uniform random int32 over the full range (config 1 put/get payloads)."""
    r = rng_for(seed, 10, pe)
    return r.integers(-2**31, 2**31, size=nelems, dtype=np.int64).astype(np.int32)


def int32_reduce_values(seed: int, pe: int, nelems: int, lo=-1000, hi=1000) -> np.ndarray:
    """Uniform integers in [lo, hi] (config 1 sum_reduce sources)."""
    r = rng_for(seed, 11, pe)
    return r.integers(lo, hi + 1, size=nelems, dtype=np.int64).astype(np.int32)


def byte_payload(seed: int, pe: int, nbytes: int) -> np.ndarray:
    """Uniform random bytes (config 2 put/get sweep, config 4 ping-pong payloads)."""
    r = rng_for(seed, 20, pe)
    return r.integers(0, 256, size=nbytes, dtype=np.uint8)


def normal_values(seed: int, pe: int, nelems: int, dtype) -> np.ndarray:
    """N(0,1) floats (config 3 float32 / float64 collectives)."""
    r = rng_for(seed, 30, pe)
    return r.standard_normal(nelems).astype(dtype)


def int64_values(seed: int, pe: int, nelems: int, bound: int = 2**20) -> np.ndarray:
    """Uniform int64 in [-bound, bound] (config 3 int64 collectives)."""
    r = rng_for(seed, 31, pe)
    return r.integers(-bound, bound + 1, size=nelems, dtype=np.int64)


def zipf_indices(seed: int, stream: int, nops: int, nwords: int, s: float = 1.1) -> np.ndarray:
    """Indices in [0, nwords) with P(rank k) proportional to k**-s, k = 1..nwords.

    Rank k maps to word k-1, so the hottest words fall on different PEs under
    round-robin placement.  Inverse-CDF sampling of one uniform per op.
    """
    r = rng_for(seed, 40, stream)
    w = np.arange(1, nwords + 1, dtype=np.float64) ** (-s)
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    u = r.random(nops)
    idx = np.searchsorted(cdf, u, side="left")
    return np.minimum(idx, nwords - 1).astype(np.int32)


def increments(seed: int, stream: int, nops: int, lo: int = 1, hi: int = 100) -> np.ndarray:
    """Uniform int64 increments in [lo, hi] (config 4 fetch_add)."""
    r = rng_for(seed, 41, stream)
    return r.integers(lo, hi + 1, size=nops, dtype=np.int64)


def jacobi_grid(seed: int, ny: int, nx: int) -> np.ndarray:
    """float64 grid: interior uniform in [0,1), outermost ring 0 (config 5)."""
    r = rng_for(seed, 50)
    g = r.random((ny, nx))
    g[0, :] = 0.0
    g[-1, :] = 0.0
    g[:, 0] = 0.0
    g[:, -1] = 0.0
    return g


def jacobi_cell_init(seed: int, ny: int, nx: int, i0: int, i1: int, j0: int, j1: int,
                     rows_per_block: int = 1024) -> np.ndarray:
    """Window [i0:i1, j0:j1] of the grid of :func:`jacobi_grid_block` without building the whole grid."""
    out = np.empty((i1 - i0, j1 - j0), dtype=np.float64)
    b0, b1 = i0 // rows_per_block, (i1 - 1) // rows_per_block
    for b in range(b0, b1 + 1):
        blk = jacobi_grid_block(seed, ny, nx, b, rows_per_block)
        lo, hi = max(i0, b * rows_per_block), min(i1, (b + 1) * rows_per_block)
        out[lo - i0:hi - i0] = blk[lo - b * rows_per_block:hi - b * rows_per_block, j0:j1]
    return out


def jacobi_grid_block(seed: int, ny: int, nx: int, block: int,
                      rows_per_block: int = 1024) -> np.ndarray:
    """Rows [block*rows_per_block, ...) of a grid drawn block by block (full-size config 5:
    each block has its own stream, so any window can be regenerated without the 2 GiB grid)."""
    r = rng_for(seed, 51, block)
    lo = block * rows_per_block
    hi = min(ny, lo + rows_per_block)
    g = r.random((hi - lo, nx))
    if lo == 0:
        g[0, :] = 0.0
    if hi == ny:
        g[-1, :] = 0.0
    g[:, 0] = 0.0
    g[:, -1] = 0.0
    return g


def message_sizes(lo_log2: int, hi_log2: int) -> list[int]:
    """Powers of two from 2**lo_log2 to 2**hi_log2 bytes inclusive."""
    return [1 << k for k in range(lo_log2, hi_log2 + 1)]


# ---- full-size inputs, drawn block by block so that any window can be regenerated ---------

BLOCK_ELEMS = 1 << 20


def _block(kind: str, seed: int, pe: int, block: int, count: int) -> np.ndarray:
    r = rng_for(seed, 60, pe, block)
    if kind == "u8":
        return r.integers(0, 256, size=count, dtype=np.uint8)
    if kind == "f32":
        return r.standard_normal(count, dtype=np.float32)
    if kind == "f64":
        return r.standard_normal(count)
    if kind == "i64":
        return r.integers(-2**20, 2**20 + 1, size=count, dtype=np.int64)
    raise ValueError(kind)


def block_values(kind: str, seed: int, pe: int, start: int, count: int) -> np.ndarray:
    """Elements [start, start+count) of PE ``pe``'s full-size source of the given kind
    ('u8' uniform bytes, 'f32'/'f64' N(0,1), 'i64' uniform in [-2^20, 2^20]).  The stream is
    defined in blocks of 2^20 elements, each with its own generator, so a window costs only
    the blocks it touches and is identical to the same range of the whole array."""
    out = []
    b = start // BLOCK_ELEMS
    pos = start
    end = start + count
    while pos < end:
        blk = _block(kind, seed, pe, b, BLOCK_ELEMS)
        lo = pos - b * BLOCK_ELEMS
        hi = min(end - b * BLOCK_ELEMS, BLOCK_ELEMS)
        out.append(blk[lo:hi])
        pos += hi - lo
        b += 1
    return np.concatenate(out) if len(out) != 1 else out[0]
