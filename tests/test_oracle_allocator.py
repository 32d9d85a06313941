"""Pins for the oracle's symmetric allocator: offsets worked out by hand for a sequence of
sizes and alignments (round-up to the alignment, 256 B by default), the same offset naming
a distinct object on every PE, exhaustion and the refusal of alignments that are not a
power of two (Section 2.3 of the paper: a symmetric object has the same offset on all PEs)."""
import numpy as np
import pytest

import oracle as orc
from oracle import Oracle


def test_offsets_of_a_hand_worked_sequence():
    o = Oracle(3, 2048)
    # cursor 0
    assert o.malloc(100) == 0                # default alignment 256: 0 is aligned; cursor 100
    assert o.malloc(1) == 256                # 100 rounds up to 256; cursor 257
    assert o.malloc(300, 64) == 320          # 257 rounds up to 5*64 = 320; cursor 620
    assert o.malloc(8, 1024) == 1024         # 620 rounds up to 1024; cursor 1032
    assert o.malloc(0, 8) == 1032            # 1032 = 129*8 is aligned; an empty object; cursor 1032
    assert o.malloc(5, 1) == 1032            # alignment 1 never moves the cursor; cursor 1037
    assert o.malloc(3, 2) == 1038            # 1037 rounds up to 1038; cursor 1041
    assert o.malloc(1007, 1) == 1041         # ends exactly at 2048
    with pytest.raises(orc.OracleError) as e:
        o.malloc(1, 1)                       # nothing left
    assert e.value.code == orc.ERR_OOM
    assert o.malloc(0, 1) == 2048            # an empty object at the very end still fits
    o.close()


def test_exhaustion_cases():
    o = Oracle(2, 1000)
    assert o.malloc(700) == 0                # cursor 700
    with pytest.raises(orc.OracleError) as e:
        o.malloc(300)                        # 768 + 300 > 1000
    assert e.value.code == orc.ERR_OOM
    with pytest.raises(orc.OracleError) as e:
        o.malloc(0, 1024)                    # 700 rounds up to 1024 > 1000
    assert e.value.code == orc.ERR_OOM
    with pytest.raises(orc.OracleError) as e:
        o.malloc(2**63, 1)                   # a size that would wrap the arithmetic
    assert e.value.code == orc.ERR_OOM
    assert o.malloc(232) == 768              # failed calls did not move the cursor; ends at 1000
    o.reset_allocator()
    assert o.malloc(1000, 1) == 0            # the whole heap again
    o.close()


@pytest.mark.parametrize("align", [0, 3, 6, 48, 255, 257, 1000])
def test_alignment_must_be_a_power_of_two(align):
    o = Oracle(1, 4096)
    with pytest.raises(orc.OracleError) as e:
        o.malloc(8, align)
    assert e.value.code == orc.ERR_ALIGN
    assert o.malloc(8, 1) == 0               # the refused call changed nothing
    o.close()


def test_one_offset_names_one_object_per_pe():
    npes, heap = 4, 4096
    o = Oracle(npes, heap)
    a = o.malloc(40)
    b = o.malloc(24, 512)
    assert (a, b) == (0, 512)
    bases = [o.ptr(0, 0, p) for p in range(npes)]
    assert len(set(bases)) == npes
    for p in range(npes):
        # translation: heap base of the PE plus the offset
        assert o.ptr(b, 24, p) - bases[p] == b
        o.view(b, 24, p)[:] = p + 1
    for p in range(npes):                    # the four copies are separate memory
        assert (o.view(b, 24, p) == p + 1).all()
        assert not o.view(a, 40, p).any()    # and the neighbouring object is untouched
    with pytest.raises(orc.OracleError):
        o.ptr(b, heap - b + 1, 0)            # a range that leaves the heap
    with pytest.raises(orc.OracleError):
        o.ptr(0, 1, npes)                    # a PE that does not exist
    assert o.ptr(heap, 0, 0) - bases[0] == heap
    o.close()
