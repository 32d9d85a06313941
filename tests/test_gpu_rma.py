"""GPU parity: symmetric heap, put/get in every collaboration level, p/g, nbi/quiet,
copy-engine path, put_signal / wait_until -- element by element against the CPU oracle
through the C ABI."""
import itertools

import numpy as np
import pytest
import torch

import oracle as orc
from paper_2409_20476_b200 import binding as B
from paper_2409_20476_b200 import inputs
from tests.gpu_util import Session, heaps_equal

pytestmark = pytest.mark.gpu

LEVELS = {"work_item": B.ISHMEMX_WORK_ITEM, "sub_group": B.ISHMEMX_SUB_GROUP,
          "work_group": B.ISHMEMX_WORK_GROUP, "work_group_bulk": B.ISHMEMX_WORK_GROUP_BULK}


def test_allocator_properties():
    with Session(3, 1 << 20, with_oracle=False) as s:
        assert B.ishmem_n_pes() == 3 and B.ishmemx_heap_bytes() == 1 << 20
        a = B.ishmem_malloc(1000)
        b = B.ishmem_malloc(1)
        c = B.ishmem_align(4096, 5000)
        assert a and b and c
        for p in (a, b, c):
            assert s.base <= p < s.base + (1 << 20) and p % 256 == 0   # inside PE 0's slice
        assert c % 4096 == 0
        spans = sorted([(a, 1000), (b, 1), (c, 5000)])
        assert all(x[0] + x[1] <= y[0] for x, y in zip(spans, spans[1:]))  # disjoint
        for pe in range(3):                                              # same offset everywhere
            assert B.ishmem_ptr(a, pe) == a + pe * (1 << 20)
        assert B.ishmem_ptr(a, 3) == 0 and B.ishmem_ptr(s.base - 1, 0) == 0
        assert B.ishmem_malloc(1 << 20) == 0                             # exhausted -> NULL
        assert B.ishmem_malloc(0) == 0
        B.ishmem_free(0)                                                 # free(NULL) is a no-op
        with pytest.raises(B.IshmemError) as e:
            B.ishmem_free(a + 256)
        assert e.value.code == B.ISHMEM_ERR_ARG
        for p in (a, b, c):
            B.ishmem_free(p)
        big = B.ishmem_malloc(1 << 20)                                   # coalesced back to one block
        assert big == s.base
        B.ishmem_free(big)
        # calloc zero-fills every PE's copy
        s.heap.fill_(0xAB)
        z = B.ishmem_calloc(100, 8)
        s.sync()
        for pe in range(3):
            off = z - s.base + pe * (1 << 20)
            assert not s.heap[off:off + 800].any()
            assert s.heap[off + 800] == 0xAB


def test_errors_and_not_initialized():
    with pytest.raises(B.IshmemError) as e:
        B.ishmem_putmem(0, 1, 1, 1, 0)
    assert e.value.code == B.ISHMEM_ERR_NOT_INITIALIZED
    with Session(2, 1 << 16, with_oracle=False) as s:
        a = B.ishmem_malloc(4096)
        priv = torch.zeros(4096, dtype=torch.uint8, device="cuda")
        for bad_pe in (-1, 2):
            with pytest.raises(B.IshmemError) as e:
                B.ishmem_putmem(0, a, priv, 16, bad_pe)
            assert e.value.code == B.ISHMEM_ERR_INVALID_PE
        with pytest.raises(B.IshmemError) as e:
            B.ishmem_putmem(0, priv, a, 16, 1)           # dest of a put must be symmetric
        assert e.value.code == B.ISHMEM_ERR_NOT_SYMMETRIC
        with pytest.raises(B.IshmemError) as e:
            B.ishmem_getmem(0, a, priv, 16, 1)           # src of a get must be symmetric
        assert e.value.code == B.ISHMEM_ERR_NOT_SYMMETRIC
        with pytest.raises(B.IshmemError) as e:
            B.ishmem_putmem(0, s.base + (1 << 16) - 8, priv, 16, 1)   # runs off the heap
        assert e.value.code == B.ISHMEM_ERR_NOT_SYMMETRIC
        with pytest.raises(B.IshmemError) as e:
            B.ishmem_int64_put(0, a + 4, priv, 1, 1)
        assert e.value.code == B.ISHMEM_ERR_ALIGN
        with pytest.raises(B.IshmemError) as e:
            B.ishmem_init(2, 1 << 16)                    # already initialised
        assert e.value.code == B.ISHMEM_ERR_ARG
        s.sync()
        assert not s.heap.any() and s.status() == 0


@pytest.mark.parametrize("level", list(LEVELS))
def test_config1_put_get_ring_all_sizes(level):
    """Config 1: 4 PEs x 16 MiB, int32 payloads 4 B..1 MiB, PE p -> (p+1)%4, put then get."""
    npes, heap = 4, 16 << 20
    with Session(npes, heap) as s:
        src, dst, back = s.malloc(1 << 20), s.malloc(1 << 20), s.malloc(1 << 20)
        threads = {"work_item": 64, "sub_group": 128, "work_group": 256, "work_group_bulk": 256}[level]
        for k, n in enumerate(inputs.message_sizes(2, 20)):
            for p in range(npes):
                src.fill(p, inputs.int32_payload(inputs.SEED_C1, p * 100 + k, n // 4))
            groups = 1 if n < 65536 else 3
            for p in range(npes):
                t = (p + 1) % npes
                B.ishmemx_putmem_on_device(p, dst.addr, src.addr, n, t, LEVELS[level], threads, groups)
                s.oracle.putmem(p, dst.ooff, s.oracle.ptr(src.ooff, n, p), n, t)
            B.ishmem_barrier_all()
            for p in range(npes):
                t = (p + 1) % npes
                B.ishmemx_getmem_on_device(p, back.addr, dst.addr, n, t, LEVELS[level], threads, groups)
                s.oracle.getmem(p, s.oracle.ptr(back.ooff, n, p), dst.ooff, n, t)
            B.ishmem_barrier_all()
        heaps_equal(s, level)
        assert s.status() == 0


@pytest.mark.parametrize("level", list(LEVELS))
def test_spmd_ring_and_all_pairs(level):
    npes, heap, n = 8, 4 << 20, 300_001
    with Session(npes, heap) as s:
        src, dst = s.malloc(n + 64), s.malloc(n + 64)
        for p in range(npes):
            src.fill(p, inputs.byte_payload(inputs.SEED_C2, p, n + 64))
        for shift in range(1, npes):          # the all-pairs pattern as permutation rounds
            B.ishmemx_putmem_spmd(dst.addr + 3, src.addr + 3, n, shift, LEVELS[level], 256, 5)
            for p in range(npes):
                s.oracle.putmem(p, dst.ooff + 3, s.oracle.ptr(src.ooff + 3, n, p), n, (p + shift) % npes)
            dst.assert_equal(f"put shift {shift}")
        B.ishmemx_getmem_spmd(src.addr + 16, dst.addr + 16, n, 3, LEVELS[level], 256, 5)
        for p in range(npes):
            s.oracle.getmem(p, s.oracle.ptr(src.ooff + 16, n, p), dst.ooff + 16, n, (p + 3) % npes)
        heaps_equal(s, level)
        assert s.status() == 0


@pytest.mark.parametrize("threads", [32, 256, 1024])
def test_spmd_grid_sized_by_the_library(threads):
    """groups = 0: one tile of threads x 128 bytes per block.  Ragged sizes around the tile size and
    misaligned, non-congruent addresses against the oracle; the heaps are compared whole."""
    npes, heap = 5, 4 << 20
    tile = threads * 128
    with Session(npes, heap) as s:
        src, dst = s.malloc(1 << 20), s.malloc(1 << 20)
        for p in range(npes):
            src.fill(p, inputs.byte_payload(inputs.SEED_C2, p, 1 << 20))
        cases = [(0, 0, 1), (0, 0, tile - 1), (0, 0, tile), (3, 3, tile + 1), (16, 5, 3 * tile + 77),
                 (1, 2, 7 * tile - 13), (0, 8, 500_000), (0, 0, 0)]
        for k, (doff, soff, n) in enumerate(cases):
            shift = 1 + k % (npes - 1)
            B.ishmemx_putmem_spmd(dst.addr + doff, src.addr + soff, n, shift, B.ISHMEMX_WORK_GROUP, threads, 0)
            for p in range(npes):
                s.oracle.putmem(p, dst.ooff + doff, s.oracle.ptr(src.ooff + soff, n, p), n, (p + shift) % npes)
            dst.assert_equal(f"put case {k}")
        B.ishmemx_getmem_spmd(src.addr + 32, dst.addr + 1, 2 * tile + 5, 2, B.ISHMEMX_WORK_GROUP, threads, 0)
        for p in range(npes):
            s.oracle.getmem(p, s.oracle.ptr(src.ooff + 32, 2 * tile + 5, p), dst.ooff + 1, 2 * tile + 5, (p + 2) % npes)
        heaps_equal(s, f"threads {threads}")
        # the host API picks the same shape by itself above 256 KiB
        B.ishmem_putmem(0, dst.addr + 7, src.addr + 7, 900_001, 3)
        s.oracle.putmem(0, dst.ooff + 7, s.oracle.ptr(src.ooff + 7, 900_001, 0), 900_001, 3)
        B.ishmem_barrier_all()
        heaps_equal(s, "host api")
        assert s.status() == 0


@pytest.mark.parametrize("level", ["work_item", "sub_group", "work_group", "work_group_bulk"])
def test_misaligned_brute_force(level):
    """Every source/destination alignment mod 16 with ragged lengths, private and symmetric
    sources, against the oracle; the heap is compared whole, so stray writes show up."""
    npes, heap = 3, 1 << 19
    with Session(npes, heap) as s:
        src, dst = s.malloc(150_000), s.malloc(150_000)
        for p in range(npes):
            src.fill(p, inputs.byte_payload(7, p, 150_000))
            dst.fill(p, inputs.byte_payload(8, p, 150_000))
        threads = {"work_item": 32, "sub_group": 64, "work_group": 96, "work_group_bulk": 160}[level]
        lens = [0, 1, 5, 15, 16, 17, 31, 33, 64, 100, 255, 1000, 4099]
        if level != "work_item":
            lens += [16384, 16385, 40_000, 100_003]     # past the TMA threshold, ragged tails
        sa = [0, 1, 4, 7, 8, 15]
        da = [0, 1, 2, 8, 9, 15]
        case = 0
        for n, so, do in itertools.product(lens, sa, da):
            if n > 4099 and (so, do) not in ((0, 0), (1, 1), (7, 7), (8, 8), (15, 15), (4, 8), (1, 2), (0, 9)):
                continue
            me, pe = case % npes, (case // 2) % npes
            case += 1
            B.ishmemx_putmem_on_device(me, dst.addr + 256 + do, src.addr + 512 + so, n, pe, LEVELS[level],
                                       threads, 1 + case % 2)
            s.oracle.putmem(me, dst.ooff + 256 + do, s.oracle.ptr(src.ooff + 512 + so, n, me), n, pe)
            B.ishmem_quiet(me)
            B.ishmem_sync_all()       # cases of different PEs overlap in dest: keep them ordered
            if case % 64 == 0:
                heaps_equal(s, f"{level} case {case}")
        heaps_equal(s, level)
        # private (non-symmetric) source and destination buffers
        priv = torch.from_numpy(inputs.byte_payload(9, 0, 70_000)).cuda()
        B.ishmemx_putmem_on_device(1, dst.addr + 5, priv[3:], 60_001, 2, LEVELS[level], threads, 2)
        s.oracle.putmem(1, dst.ooff + 5, priv[3:].cpu().numpy(), 60_001, 2)
        out = torch.zeros(70_000, dtype=torch.uint8, device="cuda")
        B.ishmemx_getmem_on_device(0, out[1:], dst.addr + 5, 60_001, 2, LEVELS[level], threads, 2)
        exp = np.zeros(60_001, dtype=np.uint8)
        s.oracle.getmem(0, exp, dst.ooff + 5, 60_001, 2)
        s.sync()
        assert np.array_equal(out[1:60_002].cpu().numpy(), exp) and out[0] == 0 and out[60_002] == 0
        heaps_equal(s, level + " private")
        assert s.status() == 0


def test_host_put_get_typed_nbi_cutover_and_copy_engine():
    npes, heap = 4, 8 << 20
    with Session(npes, heap) as s:
        src, dst = s.malloc(2 << 20), s.malloc(2 << 20)
        for p in range(npes):
            src.fill(p, inputs.byte_payload(11, p, 2 << 20))
        # blocking host put/get with automatic geometry, several sizes
        for n in (1, 8, 1000, 65_536, 1_000_003, 2 << 20):
            B.ishmem_putmem(0, dst.addr, src.addr, n, 3)
            s.oracle.putmem(0, dst.ooff, s.oracle.ptr(src.ooff, n, 0), n, 3)
            B.ishmem_getmem(2, dst.addr, src.addr, n, 1)
            s.oracle.getmem(2, s.oracle.ptr(dst.ooff, n, 2), src.ooff, n, 1)
        # typed
        B.ishmem_double_put(1, dst.addr + 8, src.addr + 16, 1000, 0)
        s.oracle.putmem(1, dst.ooff + 8, s.oracle.ptr(src.ooff + 16, 8000, 1), 8000, 0)
        B.ishmem_int32_get(3, dst.addr + 4, src.addr + 4, 77, 2)
        s.oracle.getmem(3, s.oracle.ptr(dst.ooff + 4, 308, 3), src.ooff + 4, 308, 2)
        B.ishmem_barrier_all()
        heaps_equal(s, "host put/get")
        # copy engine alone, and the cutover: above the threshold the engine is used (nbi + quiet)
        B.ishmemx_putmem_copy_engine(0, dst.addr + 100, src.addr + 7, 500_000, 1)
        s.oracle.putmem(0, dst.ooff + 100, s.oracle.ptr(src.ooff + 7, 500_000, 0), 500_000, 1)
        B.ishmemx_getmem_copy_engine(1, dst.addr + 1_000_000, src.addr, 300_000, 3)
        s.oracle.getmem(1, s.oracle.ptr(dst.ooff + 1_000_000, 300_000, 1), src.ooff, 300_000, 3)
        B.ishmemx_set_cutover(0, 4096)
        assert B.ishmemx_get_cutover(0) == 4096
        B.ishmem_putmem_nbi(2, dst.addr + 64, src.addr + 64, 700_000, 0)      # engine
        s.oracle.putmem(2, dst.ooff + 64, s.oracle.ptr(src.ooff + 64, 700_000, 2), 700_000, 0)
        B.ishmem_putmem_nbi(2, dst.addr, src.addr, 40, 3)                      # kernel
        s.oracle.putmem(2, dst.ooff, s.oracle.ptr(src.ooff, 40, 2), 40, 3)
        B.ishmem_quiet(2)
        B.ishmem_getmem(2, dst.addr + 1_500_000, dst.addr + 64, 100_000, 0)    # ordered after the nbi put
        s.oracle.getmem(2, s.oracle.ptr(dst.ooff + 1_500_000, 100_000, 2), dst.ooff + 64, 100_000, 0)
        B.ishmemx_set_cutover(0, B.SIZE_MAX)
        B.ishmem_barrier_all()
        heaps_equal(s, "engine / cutover")
        assert s.status() == 0


def test_host_cutover_is_a_band_between_two_sizes():
    """The default host-initiated cutover follows the committed size sweep: the copy engine from
    4 MiB up to (not including) 64 MiB, the tiled kernel below and above.  A kernel launch shows
    in the library's launch counter, an engine copy does not; both paths are bit-exact."""
    MiB = 1 << 20
    npes, n_max = 2, 64 * MiB
    with Session(npes, 2 * n_max + MiB) as s:
        assert B.ishmemx_get_cutover(0) == 4 * MiB and B.ishmemx_get_cutover(5) == 64 * MiB
        src, dst = s.malloc(n_max), s.malloc(n_max)
        src.fill(0, inputs.byte_payload(12, 0, n_max))
        for n, kernel in ((1 * MiB, True), (4 * MiB - 1, True), (4 * MiB, False), (16 * MiB, False),
                          (64 * MiB - 1, False), (64 * MiB, True)):
            before = B.ishmemx_launch_count()
            B.ishmem_putmem(0, dst.addr, src.addr, n, 1)
            assert (B.ishmemx_launch_count() - before == 1) == kernel, (n, kernel)
            s.oracle.putmem(0, dst.ooff, s.oracle.ptr(src.ooff, n, 0), n, 1)
            B.ishmem_quiet(0)
            dst.assert_equal(f"put of {n} bytes")
            before = B.ishmemx_launch_count()
            B.ishmem_getmem(1, src.addr, dst.addr, n, 1 - 1)      # PE 1 reads PE 0's dst (zeros) into its src
            assert (B.ishmemx_launch_count() - before == 1) == kernel, (n, kernel)
            s.oracle.getmem(1, s.oracle.ptr(src.ooff, n, 1), dst.ooff, n, 0)
        B.ishmem_barrier_all()
        src.assert_equal("gets")
        # the band can be moved and removed
        B.ishmemx_set_cutover(5, B.SIZE_MAX)
        before = B.ishmemx_launch_count()
        B.ishmem_putmem(0, dst.addr, src.addr, 64 * MiB, 1)
        assert B.ishmemx_launch_count() == before
        B.ishmemx_set_cutover(5, 8 * MiB)
        B.ishmem_putmem(0, dst.addr, src.addr, 8 * MiB, 1)
        assert B.ishmemx_launch_count() == before + 1
        B.ishmem_barrier_all()
        dst.assert_equal("after moving the band")
        assert s.status() == 0


def test_scalar_p_g():
    with Session(3, 1 << 16) as s:
        buf = s.malloc(256)
        B.ishmem_long_p(0, buf.addr + 8, -5, 2)
        s.oracle.p(buf.ooff + 8, np.int64(-5), 2)
        B.ishmem_float_p(1, buf.addr + 16, 1.5, 0)
        s.oracle.p(buf.ooff + 16, np.float32(1.5), 0)
        B.ishmem_uint8_p(2, buf.addr + 21, 200, 1)
        s.oracle.p(buf.ooff + 21, np.uint8(200), 1)
        B.ishmem_double_p(2, buf.addr + 24, 2.0 ** -40, 2)
        s.oracle.p(buf.ooff + 24, np.float64(2.0 ** -40), 2)
        heaps_equal(s, "p")
        out = np.zeros(1, dtype=np.int64)
        B.ishmem_long_g(1, out, buf.addr + 8, 2)
        assert out[0] == s.oracle.g(buf.ooff + 8, np.int64, 2) == -5
        outf = np.zeros(1, dtype=np.float32)
        B.ishmem_float_g(2, outf, buf.addr + 16, 0)
        assert outf[0] == s.oracle.g(buf.ooff + 16, np.float32, 0) == 1.5
        with pytest.raises(B.IshmemError) as e:
            B.ishmem_long_p(0, buf.addr + 4, 1, 1)
        assert e.value.code == B.ISHMEM_ERR_ALIGN


def test_put_signal_wait_until_and_bounded_timeout():
    with Session(2, 1 << 20) as s:
        data, sig = s.malloc(100_000), s.malloc(64)
        payload = inputs.byte_payload(3, 0, 100_000)
        data.fill(0, payload)
        # PE 0 sends payload + signal; PE 1's stream then waits for the signal before reading
        # (the wait is enqueued after the launch that satisfies it: nothing waits on a later launch)
        B.ishmem_putmem_signal(0, data.addr, data.addr, 40_000, sig.addr, 7, B.ISHMEM_SIGNAL_SET, 1)
        B.ishmem_uint64_wait_until(1, sig.addr, B.ISHMEM_CMP_GE, 7)
        B.ishmem_getmem(1, data.addr + 50_000, data.addr, 40_000, 1)   # runs only after the wait
        s.oracle.putmem_signal(0, data.ooff, s.oracle.ptr(data.ooff, 40_000, 0), 40_000, sig.ooff, 7,
                               orc.SIG_SET, 1)
        assert s.oracle.test(1, sig.ooff, orc.C_GE, 7)
        s.oracle.getmem(1, s.oracle.ptr(data.ooff + 50_000, 40_000, 1), data.ooff, 40_000, 1)
        B.ishmem_putmem_signal(0, data.addr, data.addr, 0, sig.addr, 5, B.ISHMEM_SIGNAL_ADD, 1)
        s.oracle.putmem_signal(0, data.ooff, s.oracle.ptr(data.ooff, 0, 0), 0, sig.ooff, 5, orc.SIG_ADD, 1)
        B.ishmem_barrier_all()
        heaps_equal(s, "put_signal")
        assert s.status() == 0
        # a wait nothing satisfies gives up after the limit and latches TIMEOUT; the context
        # stays usable
        B.ishmemx_set_wait_limit_ns(20_000_000)
        B.ishmem_uint64_wait_until(0, sig.addr + 8, B.ISHMEM_CMP_EQ, 1)
        assert s.status() == B.ISHMEM_ERR_TIMEOUT
        assert s.status() == 0                                           # cleared
        B.ishmemx_set_wait_limit_ns(2_000_000_000)
        B.ishmem_putmem(0, data.addr, data.addr, 16, 1)
        B.ishmem_barrier_all()
        assert s.status() == 0


@pytest.mark.parametrize("level", list(LEVELS))
def test_device_timed_latency_program_moves_the_data(level):
    """ishmemx_rma_latency: repeated in-kernel put/get + quiet by one collaboration unit; the
    payload must arrive exactly as the oracle's put/get says and the time must be positive."""
    npes, heap = 3, 1 << 20
    with Session(npes, heap) as s:
        src, dst = s.malloc(200_000), s.malloc(200_000)
        for p in range(npes):
            src.fill(p, inputs.byte_payload(inputs.SEED_C2, p, 200_000))
        ns = np.zeros(1)
        for n, is_get in ((8, 0), (4099, 0), (150_001, 0), (65_536, 1), (33, 1)):
            threads = {"work_item": 32, "sub_group": 64, "work_group": 128, "work_group_bulk": 256}[level]
            B.ishmemx_rma_latency(1, dst.addr + 5, src.addr + 5, n, 2, is_get, LEVELS[level], threads, 3, ns)
            assert ns[0] > 0
            if is_get:
                s.oracle.getmem(1, s.oracle.ptr(dst.ooff + 5, n, 1), src.ooff + 5, n, 2)
            else:
                s.oracle.putmem(1, dst.ooff + 5, s.oracle.ptr(src.ooff + 5, n, 1), n, 2)
            heaps_equal(s, f"{level} n={n} get={is_get}")
        with pytest.raises(B.IshmemError) as e:
            B.ishmemx_rma_latency(1, dst.addr, src.addr, 8, 7, 0, LEVELS[level], 64, 1, ns)
        assert e.value.code == B.ISHMEM_ERR_INVALID_PE
        assert s.status() == 0


def test_environment_variables_at_initialisation(monkeypatch):
    monkeypatch.setenv("ISHMEM_SYMMETRIC_SIZE", str(3 << 20))
    monkeypatch.setenv("ISHMEM_CUTOVER_PUT", "never")
    monkeypatch.setenv("ISHMEM_CUTOVER_BCAST", "always")
    monkeypatch.setenv("ISHMEM_CUTOVER_FCOLLECT", "0x10000")
    monkeypatch.setenv("ISHMEM_CUTOVER_PUT_UPTO", str(1 << 20))
    monkeypatch.setenv("ISHMEM_JACOBI_SPLIT", "columns")
    monkeypatch.setenv("ISHMEM_JACOBI_FUSE", "0")
    monkeypatch.setenv("ISHMEM_REDUCE_BULK", "1")
    B.ishmem_init(2, 0)
    try:
        # launch-shape switches: initial values from the environment, then only set_option counts
        assert B.ishmemx_get_cutover(5) == 1 << 20
        assert B.ishmemx_get_option(B.ISHMEMX_OPT_JACOBI_SPLIT) == 2
        assert B.ishmemx_get_option(B.ISHMEMX_OPT_JACOBI_FUSE) == 0
        assert B.ishmemx_get_option(B.ISHMEMX_OPT_JACOBI_WIDE) == -1
        assert B.ishmemx_get_option(B.ISHMEMX_OPT_REDUCE_BULK) == 1
        monkeypatch.setenv("ISHMEM_JACOBI_SPLIT", "rows")            # not read again
        assert B.ishmemx_get_option(B.ISHMEMX_OPT_JACOBI_SPLIT) == 2
        B.ishmemx_set_option(B.ISHMEMX_OPT_JACOBI_SPLIT, 0)
        assert B.ishmemx_get_option(B.ISHMEMX_OPT_JACOBI_SPLIT) == 0
        for opt, bad in ((B.ISHMEMX_OPT_JACOBI_SPLIT, 3), (B.ISHMEMX_OPT_JACOBI_WIDE, -2), (99, 0),
                         (B.ISHMEMX_OPT_BULK_SMEM, 100)):
            with pytest.raises(B.IshmemError) as e:
                B.ishmemx_set_option(opt, bad)
            assert e.value.code == B.ISHMEM_ERR_ARG
        assert B.ishmemx_heap_bytes() == 3 << 20 and B.ishmem_n_pes() == 2
        assert B.ishmemx_get_cutover(0) == B.SIZE_MAX and B.ishmemx_get_cutover(1) == 0
        assert B.ishmemx_get_cutover(2) == 0x10000 and B.ishmemx_get_cutover(3) == B.SIZE_MAX
        a = B.ishmem_calloc(16, 8)
        B.ishmem_int64_p(0, a + 8, -5, 1)
        out = np.zeros(1, np.int64)
        B.ishmem_int64_g(0, out, a + 8, 1)
        assert out[0] == -5
    finally:
        B.ishmem_finalize()
    monkeypatch.delenv("ISHMEM_SYMMETRIC_SIZE")
    with pytest.raises(B.IshmemError) as e:
        B.ishmem_init(2, 0)
    assert e.value.code == B.ISHMEM_ERR_ARG


@pytest.mark.parametrize("pinned,npes,n", [(True, 5, 70_001), (False, 5, 70_001), (True, 3, (20 << 20) + 12_345)])
def test_host_put_ring_with_host_buffers(pinned, npes, n):
    """The end-to-end entry point: host payloads in, ring put on the device, destinations back
    on the host -- against the oracle's puts, with pinned and with pageable host memory, and with a
    message of 20 MiB and an odd tail."""
    with Session(npes, max(1 << 19, 2 * n + (1 << 16))) as s:
        src, dst = s.malloc(n), s.malloc(n)
        hsrc = torch.from_numpy(np.concatenate([inputs.byte_payload(inputs.SEED_C2, 500 + p, n) for p in range(npes)]))
        hdst = torch.zeros(npes * n, dtype=torch.uint8)
        if pinned:
            hsrc, hdst = hsrc.pin_memory(), hdst.pin_memory()
        for level, shift in (("work_group", 1), ("work_group_bulk", 3)):
            B.ishmemx_host_put_ring(hdst.data_ptr(), hsrc.data_ptr(), dst.addr, src.addr, n, shift, LEVELS[level], 256, 2)
            for p in range(npes):
                s.oracle.view(src.ooff, n, p)[:] = hsrc[p * n:(p + 1) * n].numpy()
                s.oracle.putmem(p, dst.ooff, s.oracle.ptr(src.ooff, n, p), n, (p + shift) % npes)
            heaps_equal(s, f"host_put_ring {level}")
            for p in range(npes):
                t = (p + shift) % npes
                assert torch.equal(hdst[t * n:(t + 1) * n], hsrc[p * n:(p + 1) * n]), (level, p)
        assert s.status() == 0
