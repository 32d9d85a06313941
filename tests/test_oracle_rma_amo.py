"""Pins for the CPU oracle's RMA, signalling and atomic operations.

Each test checks the oracle against something other than itself: a
byte-at-a-time Python model on tiny heaps (brute force), identities the
OpenSHMEM semantics fix (put-then-get, put to self = local copy), library
routines the operation reduces to (bytes slicing, numpy integer wrap), and
conservation / chain invariants of atomic read-modify-writes.
"""
import itertools

import numpy as np
import pytest

import oracle as orc
from oracle import Oracle
from paper_2409_20476_b200 import inputs


def heaps_as_lists(o):
    return [bytearray(o.view(0, o.heap_bytes, p).tobytes()) for p in range(o.npes)]


def fill_pattern(o):
    for p in range(o.npes):
        v = o.view(0, o.heap_bytes, p)
        v[:] = (np.arange(o.heap_bytes) * 7 + 31 * p + 3) % 251


def test_create_zero_filled_and_translation():
    o = Oracle(3, 128)
    for p in range(3):
        assert not o.view(0, 128, p).any()
    # same offset, distinct storage per PE (Section 2.3: same layout, different values)
    bases = [o.ptr(0, 0, p) for p in range(3)]
    assert len(set(bases)) == 3
    for p in range(3):
        assert o.ptr(40, 8, p) - bases[p] == 40
    with pytest.raises(orc.OracleError):
        o.ptr(121, 8, 0)
    with pytest.raises(orc.OracleError):
        o.ptr(0, 1, 3)
    assert o.ptr(128, 0, 2) - bases[2] == 128  # empty range at the end is legal


def test_put_brute_force_tiny_heaps():
    """All (src_off, dst_off, len, my_pe, pe) on 3 PEs x 64-byte heaps vs a Python byte model."""
    o = Oracle(3, 64)
    offs = [0, 1, 3, 8, 15, 16, 17, 31, 33, 48]
    lens = [0, 1, 2, 3, 4, 7, 8, 15, 16, 17, 31]
    for so, do, n, me, pe in itertools.product(offs, offs, lens, range(3), range(3)):
        if so + n > 64 or do + n > 64:
            continue
        if me == pe and not (so + n <= do or do + n <= so):
            continue  # overlapping local copy is undefined
        fill_pattern(o)
        model = heaps_as_lists(o)
        for k in range(n):  # byte-at-a-time definition
            model[pe][do + k] = model[me][so + k]
        o.putmem(me, do, o.ptr(so, n, me), n, pe)
        got = heaps_as_lists(o)
        assert got == model, (so, do, n, me, pe)


def test_get_brute_force_tiny_heaps():
    o = Oracle(2, 64)
    offs = [0, 1, 5, 16, 18, 32, 47]
    lens = [0, 1, 3, 8, 16, 17]
    for so, do, n, me, pe in itertools.product(offs, offs, lens, range(2), range(2)):
        if so + n > 64 or do + n > 64:
            continue
        if me == pe and not (so + n <= do or do + n <= so):
            continue
        fill_pattern(o)
        model = heaps_as_lists(o)
        for k in range(n):
            model[me][do + k] = model[pe][so + k]
        o.getmem(me, o.ptr(do, n, me), so, n, pe)
        assert heaps_as_lists(o) == model, (so, do, n, me, pe)


@pytest.mark.parametrize("n", [0, 1, 13, 4096, 100003])
def test_put_then_get_identity_and_memcpy(n):
    o = Oracle(4, 1 << 18)
    src = inputs.byte_payload(1, 0, n)
    before = [o.view(0, o.heap_bytes, p).copy() for p in range(4)]
    o.putmem(0, 777, src, n, 2)               # private source -> PE 2
    back = np.zeros(n, dtype=np.uint8)
    o.getmem(3, back, 777, n, 2)              # PE 3 reads it back
    assert back.tobytes() == src.tobytes()     # put-then-get identity
    # equals a bytes slice assignment (library routine), nothing else touched
    exp = before[2].copy()
    exp[777:777 + n] = src
    assert np.array_equal(o.view(0, o.heap_bytes, 2), exp)
    for p in (0, 1, 3):
        assert np.array_equal(o.view(0, o.heap_bytes, p), before[p])


def test_put_to_self_is_local_copy_and_get_then_put():
    o = Oracle(2, 4096)
    data = inputs.byte_payload(1, 1, 1000)
    o.view(0, 1000, 1)[:] = data
    o.putmem(1, 2000, o.ptr(0, 1000, 1), 1000, 1)
    assert np.array_equal(o.view(2000, 1000, 1), data)
    # get from PE 1 into PE 0, then put back to another place on PE 1: same bytes
    o.getmem(0, o.ptr(100, 1000, 0), 2000, 1000, 1)
    o.putmem(0, 3000, o.ptr(100, 1000, 0), 1000, 1)
    assert np.array_equal(o.view(3000, 1000, 1), data)


def test_rma_rejects_bad_pe_and_range():
    o = Oracle(2, 256)
    buf = np.zeros(300, dtype=np.uint8)
    for bad in (-1, 2):
        with pytest.raises(orc.OracleError) as e:
            o.putmem(0, 0, buf, 8, bad)
        assert e.value.code == orc.ERR_INVALID_PE
    with pytest.raises(orc.OracleError) as e:
        o.putmem(0, 250, buf, 8, 1)
    assert e.value.code == orc.ERR_NOT_SYMMETRIC
    with pytest.raises(orc.OracleError) as e:
        o.getmem(0, buf, 1, 256, 1)
    assert e.value.code == orc.ERR_NOT_SYMMETRIC
    assert not o.view(0, 256, 0).any() and not o.view(0, 256, 1).any()


@pytest.mark.parametrize("dtype", [np.int32, np.int64, np.float32, np.float64, np.uint8])
def test_scalar_p_g(dtype):
    o = Oracle(3, 256)
    val = np.array([113], dtype=dtype)[0]
    es = np.dtype(dtype).itemsize
    o.p(8 * 3, val, 2)
    raw = o.view(24, es, 2).tobytes()
    assert raw == np.array([val]).tobytes()          # little-endian image of the value
    assert o.g(24, dtype, 2) == val
    assert not o.view(0, 256, 0).any() and not o.view(0, 256, 1).any()
    if es > 1:
        with pytest.raises(orc.OracleError) as e:
            o.p(1, val, 0)
        assert e.value.code == orc.ERR_ALIGN


def test_put_signal_set_add_and_order():
    o = Oracle(2, 1024)
    payload = inputs.byte_payload(3, 0, 100)
    o.putmem_signal(0, 64, payload, 100, 512, 5, orc.SIG_SET, 1)
    assert np.array_equal(o.view(64, 100, 1), payload)
    assert o.view(512, 8, 1, np.uint64)[0] == 5
    o.putmem_signal(0, 64, payload, 0, 512, 2**64 - 3, orc.SIG_ADD, 1)  # wraps mod 2^64
    assert o.view(512, 8, 1, np.uint64)[0] == 2
    assert o.view(512, 8, 0, np.uint64)[0] == 0       # only the target's word moves
    # a failing payload must not touch the signal word
    with pytest.raises(orc.OracleError):
        o.putmem_signal(0, 1000, payload, 100, 512, 9, orc.SIG_SET, 1)
    assert o.view(512, 8, 1, np.uint64)[0] == 2


def test_wait_until_comparisons_truth_table():
    o = Oracle(1, 64)
    o.view(8, 8, 0, np.uint64)[0] = 10
    table = {orc.C_EQ: (False, True, False), orc.C_NE: (True, False, True),
             orc.C_GT: (True, False, False), orc.C_GE: (True, True, False),
             orc.C_LT: (False, False, True), orc.C_LE: (False, True, True)}
    for cmp, exp in table.items():
        got = tuple(o.test(0, 8, cmp, v) for v in (9, 10, 11))
        assert got == exp, cmp
    # unsigned comparison
    o.view(8, 8, 0, np.uint64)[0] = 2**63
    assert o.test(0, 8, orc.C_GT, 1)


def test_atomic_ops_single():
    o = Oracle(2, 64)
    t = 16
    assert o.atomic(orc.A_FETCH_ADD, 8, t, 5, 0, 1) == 0
    assert o.atomic(orc.A_FETCH_ADD, 8, t, 2**64 - 1, 0, 1) == 5        # add -1, wraps
    assert o.atomic(orc.A_FETCH, 8, t, 0, 0, 1) == 4
    assert o.atomic(orc.A_COMPARE_SWAP, 8, t, 99, 3, 1) == 4             # cond fails
    assert o.view(t, 8, 1, np.uint64)[0] == 4
    assert o.atomic(orc.A_COMPARE_SWAP, 8, t, 99, 4, 1) == 4             # cond holds
    assert o.view(t, 8, 1, np.uint64)[0] == 99
    assert o.atomic(orc.A_SWAP, 8, t, 7, 0, 1) == 99
    o.atomic(orc.A_INC, 8, t, 0, 0, 1)
    assert o.atomic(orc.A_FETCH_INC, 8, t, 0, 0, 1) == 8
    o.atomic(orc.A_SET, 8, t, 0b1100, 0, 1)
    assert o.atomic(orc.A_FETCH_AND, 8, t, 0b1010, 0, 1) == 0b1100
    assert o.atomic(orc.A_FETCH_OR, 8, t, 0b0001, 0, 1) == 0b1000
    assert o.atomic(orc.A_FETCH_XOR, 8, t, 0b1111, 0, 1) == 0b1001
    assert o.view(t, 8, 1, np.uint64)[0] == 0b0110
    assert not o.view(0, 64, 0).any()                                    # PE 0 untouched
    # 32-bit: wraps at 2^32 and leaves the neighbouring word alone
    o.view(32, 4, 0, np.uint32)[0] = 2**32 - 1
    o.view(36, 4, 0, np.uint32)[0] = 77
    assert o.atomic(orc.A_FETCH_ADD, 4, 32, 2, 0, 0) == 2**32 - 1
    assert o.view(32, 4, 0, np.uint32)[0] == 1 and o.view(36, 4, 0, np.uint32)[0] == 77
    with pytest.raises(orc.OracleError) as e:
        o.atomic(orc.A_FETCH_ADD, 8, 4, 1, 0, 0)
    assert e.value.code == orc.ERR_ALIGN


def chain_check(word, inc, fetched, init=0):
    """Per word: sorted by fetched value, fetched[k+1] == fetched[k] + inc[k] from `init`."""
    order = np.lexsort((fetched, word))
    w, f, i = word[order], fetched[order], inc[order]
    start = np.r_[True, w[1:] != w[:-1]]
    assert np.all(f[start] == init)
    cont = ~start[1:]
    assert np.all((f[1:] == f[:-1] + i[:-1])[cont])


def test_fetch_add_batch_conservation_and_chain():
    npes, nwords, nops = 4, 64, 20000
    o = Oracle(npes, 4096)
    word = inputs.zipf_indices(3, 0, nops, nwords)
    inc = inputs.increments(3, 0, nops)
    fetched = o.fetch_add_batch(256, word, inc)
    # final table = numpy scatter-add of the increments (library routine), placed round-robin
    exp = np.zeros(nwords, dtype=np.int64)
    np.add.at(exp, word, inc)
    for w in range(nwords):
        assert o.view(256 + 8 * (w // npes), 8, w % npes, np.int64)[0] == exp[w]
    total = sum(int(o.view(256, 8 * (nwords // npes), p, np.int64).sum()) for p in range(npes))
    assert total == int(inc.sum())                        # conservation
    chain_check(word, inc, fetched)
    # sequential order: fetched value = sum of earlier increments on the same word
    seen = np.zeros(nwords, dtype=np.int64)
    for k in range(2000):
        assert fetched[k] == seen[word[k]]
        seen[word[k]] += inc[k]


def test_zipf_generator_shape():
    idx = inputs.zipf_indices(3, 1, 200000, 4096)
    assert idx.min() >= 0 and idx.max() < 4096
    freq = np.bincount(idx, minlength=4096) / len(idx)
    h = (np.arange(1, 4097) ** -1.1).sum()
    assert abs(freq[0] - 1 / h) < 0.01                    # P(rank 1) = 1/H
    assert abs(freq[1] - 2 ** -1.1 / h) < 0.01


def test_compare_swap_batch_claim_semantics():
    npes, nwords, nops = 4, 32, 5000
    o = Oracle(npes, 1024)
    word = inputs.zipf_indices(3, 2, nops, nwords)
    cond = np.zeros(nops, dtype=np.int64)
    value = np.arange(1, nops + 1, dtype=np.int64)        # op id + 1
    fetched = o.compare_swap_batch(0, word, cond, value)
    for w in np.unique(word):
        ops = np.nonzero(word == w)[0]
        winner = ops[0]                                    # sequential schedule: first op wins
        assert fetched[winner] == 0
        assert np.all(fetched[ops[1:]] == winner + 1)
        assert o.view(8 * (w // npes), 8, w % npes, np.int64)[0] == winner + 1
