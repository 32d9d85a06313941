"""GPU parity and behaviour of the reverse-offload ring: device code posts requests to the
host proxy thread, which starts the copy engine; results must equal the oracle's put/get."""
import numpy as np
import pytest
import torch

from paper_2409_20476_b200 import binding as B
from paper_2409_20476_b200 import inputs
from tests.gpu_util import Session, heaps_equal

pytestmark = pytest.mark.gpu


def stats():
    served, copies, memops = np.zeros(1, np.uint64), np.zeros(1, np.uint64), np.zeros(1, np.int32)
    B.ishmemx_proxy_stats(served, copies, memops)
    return int(served[0]), int(copies[0]), int(memops[0])


def test_engine_level_needs_a_running_proxy():
    with Session(2, 1 << 16) as s:
        a, b = s.malloc(4096), s.malloc(4096)
        with pytest.raises(B.IshmemError) as e:
            B.ishmemx_putmem_on_device(0, b.addr, a.addr, 4096, 1, B.ISHMEMX_WORK_GROUP_ENGINE, 64, 1)
        assert e.value.code == B.ISHMEM_ERR_ARG
        with pytest.raises(B.IshmemError):
            B.ishmemx_ring_benchmark(0, 1, 1, 1, None, None)
        assert s.status() == 0


def test_device_initiated_engine_put_get_match_the_oracle():
    """Every work-group posts its slice as one request (non-blocking) and quiets; sizes from 1
    byte to several hundred KiB, odd offsets on both sides (the engine takes any alignment)."""
    npes, heap = 4, 2 << 20
    with Session(npes, heap) as s:
        src, dst = s.malloc(400_000), s.malloc(400_000)
        for p in range(npes):
            src.fill(p, inputs.byte_payload(inputs.SEED_C2, p, 400_000))
        B.ishmemx_proxy_start()
        try:
            expect = 0
            for k, (n, groups, slices) in enumerate(((1, 1, 1), (8, 1, 1), (4099, 2, 2), (65_536, 1, 1),
                                                     (333_337, 3, 3))):
                so, do = 3 + k, 11 + 2 * k
                for p in range(npes):
                    t = (p + 1) % npes
                    B.ishmemx_putmem_on_device(p, dst.addr + do, src.addr + so, n, t, B.ISHMEMX_WORK_GROUP_ENGINE,
                                               128, groups)
                    s.oracle.putmem(p, dst.ooff + do, s.oracle.ptr(src.ooff + so, n, p), n, t)
                    expect += slices
                B.ishmem_barrier_all()
                heaps_equal(s, f"engine put n={n}")
                for p in range(npes):
                    t = (p + 2) % npes
                    B.ishmemx_getmem_on_device(p, src.addr + do, dst.addr + so, n, t, B.ISHMEMX_WORK_GROUP_ENGINE,
                                               64, groups)
                    s.oracle.getmem(p, s.oracle.ptr(src.ooff + do, n, p), dst.ooff + so, n, t)
                    expect += slices
                B.ishmem_barrier_all()
                heaps_equal(s, f"engine get n={n}")
            served, copies, _ = stats()
            assert copies == expect and served == expect
            # blocking form, timed inside the kernel: request, wait for the reply, quiet
            ns = np.zeros(1)
            B.ishmemx_rma_latency(0, dst.addr, src.addr, 100_000, 3, 0, B.ISHMEMX_WORK_GROUP_ENGINE, 64, 5, ns)
            s.oracle.putmem(0, dst.ooff, s.oracle.ptr(src.ooff, 100_000, 0), 100_000, 3)
            heaps_equal(s, "blocking engine put")
            assert ns[0] > 0 and stats()[1] == expect + 5
            assert s.status() == 0
        finally:
            B.ishmemx_proxy_stop()


def test_cutover_inside_the_work_group_calls():
    """With the work-group cutover set, ishmemx_putmem_work_group hands large slices to the
    engine and keeps small ones on loads and stores; put_signal above the cutover delivers
    payload and signal in the engine's stream order."""
    npes, heap = 3, 2 << 20
    with Session(npes, heap) as s:
        src, dst, sig = s.malloc(300_000), s.malloc(300_000), s.malloc(64)
        for p in range(npes):
            src.fill(p, inputs.byte_payload(inputs.SEED_C2, 7 + p, 300_000))
        B.ishmemx_proxy_start()
        try:
            B.ishmemx_set_cutover(3, 32 << 10)
            assert B.ishmemx_get_cutover(3) == 32 << 10
            for n, engine_copies in ((1000, 0), (299_999, 2), (20_000, 0)):
                before = stats()[1]
                B.ishmemx_putmem_on_device(0, dst.addr + 1, src.addr + 1, n, 2, B.ISHMEMX_WORK_GROUP, 256, 2)
                s.oracle.putmem(0, dst.ooff + 1, s.oracle.ptr(src.ooff + 1, n, 0), n, 2)
                B.ishmem_barrier_all()
                heaps_equal(s, f"cutover put n={n}")
                assert stats()[1] - before == engine_copies
            # hybrid: the group copies the first 20000 bytes (rounded down to 19968) itself
            B.ishmemx_set_cutover(4, 20_000)
            assert B.ishmemx_get_cutover(4) == 20_000
            for n in (299_999, 40_000, 19_000):
                before = stats()[1]
                B.ishmemx_putmem_on_device(1, dst.addr + 7, src.addr + 7, n, 0, B.ISHMEMX_WORK_GROUP, 128, 1)
                s.oracle.putmem(1, dst.ooff + 7, s.oracle.ptr(src.ooff + 7, n, 1), n, 0)
                B.ishmemx_getmem_on_device(2, src.addr + 9, dst.addr + 9, n, 0, B.ISHMEMX_WORK_GROUP, 128, 1)
                s.oracle.getmem(2, s.oracle.ptr(src.ooff + 9, n, 2), dst.ooff + 9, n, 0)
                B.ishmem_barrier_all()
                heaps_equal(s, f"hybrid put/get n={n}")
                assert stats()[1] - before == (2 if n >= 32 << 10 else 0)
            B.ishmemx_set_cutover(4, 0)
            # in-kernel ping-pong with every put_signal going through the engine
            B.ishmemx_set_cutover(3, 0)
            rtt, bad = np.zeros(1), np.zeros(1, dtype=np.uint64)
            before = stats()[1]
            B.ishmemx_pingpong(0, 1, dst.addr, sig.addr, 4096, 20, 128, rtt, bad)
            assert bad[0] == 0 and rtt[0] > 0
            assert stats()[1] - before == 40
            B.ishmemx_set_cutover(3, B.SIZE_MAX)
            assert s.status() == 0
        finally:
            B.ishmemx_proxy_stop()
        # after the proxy has stopped the same call is plain loads and stores again
        B.ishmemx_putmem_on_device(1, dst.addr, src.addr, 100_000, 0, B.ISHMEMX_WORK_GROUP, 256, 1)
        B.ishmem_barrier_all()
        assert torch.equal(dst.gpu(0)[:100_000], src.gpu(1)[:100_000])
        assert s.status() == 0


def test_ring_round_trip_and_request_rate():
    with Session(2, 1 << 16, with_oracle=False) as s:
        B.ishmemx_proxy_start()
        try:
            rtt, rate = np.zeros(1), np.zeros(1)
            B.ishmemx_ring_benchmark(0, 1, 1, 500, rtt, None)
            assert 200.0 < rtt[0] < 1e6                      # nanoseconds; a PCIe round trip
            B.ishmemx_ring_benchmark(1, 32, 128, 200, None, rate)   # 819200 requests through a ring of 8192: flow control
            assert rate[0] > 1e5
            served, copies, _ = stats()
            assert served == 500 + 32 * 128 * 200 and copies == 0
            print(f"ring: round trip {rtt[0]:.0f} ns, {rate[0] / 1e6:.2f} M requests/s")
            assert s.status() == 0
        finally:
            B.ishmemx_proxy_stop()


def test_cutover_tuned_from_measurement():
    """ishmemx_tune_cutover times both paths and installs its pick; transfers stay correct on
    both sides of it."""
    npes, heap = 2, 40 << 20
    with Session(npes, heap) as s:
        src, dst = s.malloc(3 << 20), s.malloc(3 << 20)
        B.ishmemx_proxy_start()
        try:
            chosen = np.zeros(1, np.uint64)
            for which, threads in ((0, 0), (3, 256)):
                B.ishmemx_tune_cutover(which, threads, 16 << 20, chosen)
                pick = int(chosen[0])
                assert pick == B.SIZE_MAX or (4096 <= pick <= 16 << 20 and pick & (pick - 1) == 0)
                assert B.ishmemx_get_cutover(which) == pick
                if which == 0:      # the host band: its upper end is a larger size tried, or open
                    upto = B.ishmemx_get_cutover(5)
                    assert upto == B.SIZE_MAX or (pick < upto <= 16 << 20 and upto & (upto - 1) == 0)
                    print(f"tuned host band up to {'the top' if upto == B.SIZE_MAX else upto}")
                print(f"tuned cutover[{which}] = {'never' if pick == B.SIZE_MAX else pick}")
            with pytest.raises(B.IshmemError) as e:
                B.ishmemx_tune_cutover(0, 0, 1 << 30, None)          # no room for the temporaries
            assert e.value.code == B.ISHMEM_ERR_OOM
            for p in range(npes):
                src.fill(p, inputs.byte_payload(inputs.SEED_C2, 30 + p, 3 << 20))
            for n in (5000, 3 << 20):
                B.ishmem_putmem(0, dst.addr, src.addr, n, 1)
                s.oracle.putmem(0, dst.ooff, s.oracle.ptr(src.ooff, n, 0), n, 1)
                B.ishmemx_putmem_on_device(1, dst.addr, src.addr, n, 0, B.ISHMEMX_WORK_GROUP, 256, 1)
                s.oracle.putmem(1, dst.ooff, s.oracle.ptr(src.ooff, n, 1), n, 0)
                B.ishmem_barrier_all()
                dst.assert_equal(f"after tuning n={n}")
            assert s.status() == 0
        finally:
            B.ishmemx_proxy_stop()


def test_many_work_groups_post_at_once():
    """296 work-groups (37 per PE) each post one slice of an 8 MiB message at the same time and
    quiet on their PE's completion counter; ring pattern, whole output checked on the device,
    twice in a row."""
    npes, n = 8, 8 << 20
    with Session(npes, 2 * n + (1 << 20), with_oracle=False) as s:
        src, dst = s.malloc(n), s.malloc(n)
        for p in range(npes):
            src.gpu(p).copy_(torch.from_numpy(inputs.block_values("u8", inputs.SEED_C2, p, 0, n)))
        s.sync()
        B.ishmemx_proxy_start()
        try:
            for shift in (1, 3):
                B.ishmemx_putmem_spmd(dst.addr, src.addr, n, shift, B.ISHMEMX_WORK_GROUP_ENGINE, 64, 37)
            s.sync()
            for p in range(npes):
                assert torch.equal(dst.gpu((p + 3) % npes), src.gpu(p)), p
            assert stats()[1] == 2 * 37 * npes
            assert s.status() == 0
        finally:
            B.ishmemx_proxy_stop()
