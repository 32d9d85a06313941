"""GPU parity of remote atomics and of the put_signal / wait_until ping-pong."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2409_20476_b200 import binding as B
from paper_2409_20476_b200 import inputs
from tests.gpu_util import Session, heaps_equal
from tests.test_oracle_rma_amo import chain_check

pytestmark = pytest.mark.gpu


def test_host_initiated_atomics_all_ops():
    with Session(3, 1 << 16) as s:
        t = s.malloc(256)
        seq = [("fetch_add", 5), ("add", 7), ("fetch_inc", None), ("inc", None), ("fetch", None),
               ("set", 0b1100), ("fetch_and", 0b1010), ("fetch_or", 1), ("fetch_xor", 0b1111),
               ("swap", 99), ("compare_swap", (98, 1)), ("compare_swap", (99, 1)), ("fetch_add", -3),
               ("or", 0b110000), ("and", 0b111100), ("xor", 0b101010), ("fetch", None)]
        omap = {"fetch_add": orc.A_FETCH_ADD, "add": orc.A_ADD, "fetch_inc": orc.A_FETCH_INC,
                "inc": orc.A_INC, "fetch": orc.A_FETCH, "set": orc.A_SET, "fetch_and": orc.A_FETCH_AND,
                "fetch_or": orc.A_FETCH_OR, "fetch_xor": orc.A_FETCH_XOR, "swap": orc.A_SWAP,
                "compare_swap": orc.A_COMPARE_SWAP,
                # the non-fetching bitwise forms change memory as the fetching ones do
                "and": orc.A_FETCH_AND, "or": orc.A_FETCH_OR, "xor": orc.A_FETCH_XOR}
        for tname, npd, width in (("int64", np.int64, 8), ("uint64", np.uint64, 8), ("int32", np.int32, 4),
                                  ("uint32", np.uint32, 4)):
            addr, ooff = t.addr + 64, t.ooff + 64
            for i, (op, arg) in enumerate(seq):
                me, pe = i % 3, (i + 1) % 3 if op != "fetch" else 1
                pe = 1                                     # one target word, issued by every PE in turn
                if tname.startswith("u") and isinstance(arg, int) and arg < 0:
                    arg = arg % (1 << (8 * width))
                f = getattr(B, f"ishmem_{tname}_atomic_{op}")
                out = np.zeros(1, dtype=npd)
                if op in ("add", "set", "and", "or", "xor"):
                    f(me, addr, arg, pe)
                    s.oracle.atomic(omap[op], width, ooff, arg, 0, pe)
                elif op == "inc":
                    f(me, addr, pe)
                    s.oracle.atomic(omap[op], width, ooff, 0, 0, pe)
                elif op in ("fetch", "fetch_inc"):
                    f(me, out, addr, pe)
                    exp = s.oracle.atomic(omap[op], width, ooff, 0, 0, pe)
                    assert int(out.view(np.uint64 if width == 8 else np.uint32)[0]) == exp, (tname, op)
                elif op == "compare_swap":
                    f(me, out, addr, arg[0], arg[1], pe)
                    exp = s.oracle.atomic(omap[op], width, ooff, arg[1], arg[0], pe)
                    assert int(out.view(np.uint64 if width == 8 else np.uint32)[0]) == exp, (tname, op)
                else:
                    f(me, out, addr, arg, pe)
                    exp = s.oracle.atomic(omap[op], width, ooff, arg, 0, pe)
                    assert int(out.view(np.uint64 if width == 8 else np.uint32)[0]) == exp, (tname, op)
                B.ishmem_barrier_all()
            heaps_equal(s, tname)
            t.fill(1, np.zeros(256, np.uint8))
        with pytest.raises(B.IshmemError) as e:
            B.ishmem_int64_atomic_add(0, t.addr + 4, 1, 1)
        assert e.value.code == B.ISHMEM_ERR_ALIGN


@pytest.mark.parametrize("aggregate", [0, 1, 2])
@pytest.mark.parametrize("nops,nwords", [(100_003, 257), (1 << 22, 4096)])
def test_config4_fetch_add_batch(nops, nwords, aggregate):
    """Config 4: 16 PEs, Zipf(1.1) targets spread round-robin over PEs, increments in
    [1,100].  Final table: bit-exact.  Fetched values: any linearisation is correct, so
    check the per-word chain invariant instead of the oracle's particular order."""
    npes = 16
    with Session(npes, 1 << 16) as s:
        table = s.malloc(8 * ((nwords + npes - 1) // npes))
        word = inputs.zipf_indices(inputs.SEED_C4, 0, nops, nwords)
        inc = inputs.increments(inputs.SEED_C4, 0, nops)
        d_word, d_inc = torch.from_numpy(word).cuda(), torch.from_numpy(inc).cuda()
        d_fetched = torch.full((nops,), -1, dtype=torch.int64, device="cuda")
        B.ishmemx_int64_atomic_fetch_add_batch(table.addr, d_word, d_inc, d_fetched, nops, 256, aggregate)
        s.oracle.fetch_add_batch(table.ooff, word, inc)
        heaps_equal(s, "fetch_add table")
        fetched = d_fetched.cpu().numpy()
        chain_check(word, inc, fetched)
        total = sum(int(table.read(p, np.int64).sum()) for p in range(npes))
        assert total == int(inc.sum())
        assert s.status() == 0


@pytest.mark.parametrize("aggregate", [0, 1])
def test_config4_compare_swap_batch(aggregate):
    """2^20 compare_swap ops on 1024 words.  (i) claim: every op tries 0 -> id+1; exactly one
    op per touched word wins and everybody else sees the winner.  (ii) a CAS that cannot
    succeed leaves the table alone (bit-exact against the oracle)."""
    npes, nwords, nops = 16, 1024, 1 << 20
    with Session(npes, 1 << 16) as s:
        table = s.malloc(8 * nwords // npes)
        word = inputs.zipf_indices(inputs.SEED_C4, 1, nops, nwords)
        cond = np.zeros(nops, dtype=np.int64)
        value = np.arange(1, nops + 1, dtype=np.int64)
        d = [torch.from_numpy(a).cuda() for a in (word, cond, value)]
        d_fetched = torch.full((nops,), -1, dtype=torch.int64, device="cuda")
        B.ishmemx_int64_atomic_compare_swap_batch(table.addr, d[0], d[1], d[2], d_fetched, nops, 256, aggregate)
        s.sync()
        fetched = d_fetched.cpu().numpy()
        final = np.zeros(nwords, dtype=np.int64)
        for p in range(npes):
            final[p::npes] = table.read(p, np.int64)
        touched = np.unique(word)
        winners = np.nonzero(fetched == 0)[0]
        assert np.array_equal(np.sort(word[winners]), touched)          # exactly one winner per word
        win_of = np.zeros(nwords, dtype=np.int64)
        win_of[word[winners]] = winners + 1
        losers = fetched != 0
        assert np.array_equal(fetched[losers], win_of[word[losers]])    # losers saw the winner
        assert np.array_equal(final[touched], win_of[touched])
        untouched = np.setdiff1d(np.arange(nwords), touched)
        assert not final[untouched].any()
        # (ii) deterministic case: bring both sides to the same table, then impossible conditions
        for p in range(npes):
            table.fill(p, final[p::npes].copy())
        cond2 = np.full(nops, -1, dtype=np.int64)
        d_cond2 = torch.from_numpy(cond2).cuda()
        B.ishmemx_int64_atomic_compare_swap_batch(table.addr, d[0], d_cond2, d[2], d_fetched, nops, 512, aggregate)
        exp_fetched = s.oracle.compare_swap_batch(table.ooff, word, cond2, value)
        heaps_equal(s, "cas no-op")
        assert np.array_equal(d_fetched.cpu().numpy(), exp_fetched)
        assert s.status() == 0


@pytest.mark.parametrize("threads", [32, 256, 1024])
def test_config4_pingpong(threads):
    """put_signal / wait_until ping-pong, payloads 8 B..64 KiB between PE pairs: the payload
    is visible whenever its signal is (no stamp mismatches), and ends up bit-exact."""
    with Session(16, 1 << 18) as s:
        data, sig = s.malloc(1 << 16), s.malloc(64)
        for n in inputs.message_sizes(3, 16):
            for (a, b) in ((0, 1), (14, 15), (3, 9)):
                payload = inputs.byte_payload(inputs.SEED_C4, a, n)
                data.fill(a, payload)
                data.fill(b, np.zeros(n, np.uint8))
                sig.fill(a, np.zeros(64, np.uint8))
                sig.fill(b, np.zeros(64, np.uint8))
                rtt, bad = np.zeros(1), np.zeros(1, dtype=np.uint64)
                rounds = 200
                B.ishmemx_pingpong(a, b, data.addr, sig.addr, n, rounds, threads, rtt, bad)
                assert bad[0] == 0 and rtt[0] > 0
                # oracle: the last round's payload (stamped with the round number) sits on both
                # sides, both signal words equal the round count
                last = payload.copy()
                last[:8] = np.frombuffer(np.uint64(rounds).tobytes(), np.uint8)
                if n >= 16:
                    last[-8:] = np.frombuffer(np.uint64(rounds).tobytes(), np.uint8)
                data.cpu(a)[:n] = last
                s.oracle.putmem_signal(a, data.ooff, s.oracle.ptr(data.ooff, n, a), n, sig.ooff, rounds,
                                       orc.SIG_SET, b)
                s.oracle.putmem_signal(b, data.ooff, s.oracle.ptr(data.ooff, n, b), n, sig.ooff, rounds,
                                       orc.SIG_SET, a)
                assert s.oracle.test(a, sig.ooff, orc.C_GE, rounds) and s.oracle.test(b, sig.ooff, orc.C_GE, rounds)
        heaps_equal(s, "pingpong")
        assert s.status() == 0
        with pytest.raises(B.IshmemError):
            B.ishmemx_pingpong(2, 2, data.addr, sig.addr, 8, 1, 32, None, None)


def test_pingpong_100k_rounds_no_signal_overtakes_its_payload():
    """Memory-model soak: 10^5 round trips at every payload size 8 B..64 KiB; each round stamps
    its number into the first and last word of the payload, and the receiver counts stamps that
    do not match the signalled round."""
    with Session(2, 1 << 18, with_oracle=False) as s:
        data, sig = s.malloc(1 << 16), s.malloc(64)
        rtt, bad = np.zeros(1), np.zeros(1, dtype=np.uint64)
        for n in inputs.message_sizes(3, 16):
            B.ishmem_uint64_p(0, sig.addr, 0, 0)
            B.ishmem_uint64_p(1, sig.addr, 0, 1)
            B.ishmemx_pingpong(0, 1, data.addr, sig.addr, n, 100_000, 256, rtt, bad)
            assert bad[0] == 0, (n, int(bad[0]))
            assert sig.read(0, np.uint64)[0] == 100_000 and sig.read(1, np.uint64)[0] == 100_000
        assert s.status() == 0


@pytest.mark.parametrize("aggregate", [0, 1])
def test_compare_swap_token_passing_is_linearisable(aggregate):
    """Op k tries CAS(word, k, k+1) on its word, for k = 0..K-1 in a shuffled order, several
    words at once.  Whatever the interleaving, an op can only succeed when the word holds exactly
    k, so the successful ops of a word must be 0..m-1 (m = final value), each of them must have
    fetched its own k, and every failed op must have fetched something else."""
    npes, nwords, K = 16, 48, 4096
    rng = inputs.rng_for(inputs.SEED_C4, 77)
    word = np.repeat(np.arange(nwords, dtype=np.int32), K)
    k = np.tile(np.arange(K, dtype=np.int64), nwords)
    perm = rng.permutation(word.size)
    word, k = word[perm].copy(), k[perm].copy()
    with Session(npes, 1 << 16, with_oracle=False) as s:
        table = s.malloc(8 * nwords // npes)
        d = [torch.from_numpy(a).cuda() for a in (word, k, k + 1)]
        fetched = torch.full((word.size,), -1, dtype=torch.int64, device="cuda")
        for _ in range(3):                                  # later passes continue where the word stands
            B.ishmemx_int64_atomic_compare_swap_batch(table.addr, d[0], d[1], d[2], fetched, word.size, 1024, aggregate)
            s.sync()
            f = fetched.cpu().numpy()
            final = np.zeros(nwords, dtype=np.int64)
            for p in range(npes):
                final[p::npes] = table.read(p, np.int64)
            ok = f == k
            for w in range(nwords):
                sel = word == w
                won = np.sort(k[sel][ok[sel]])
                assert won.size == 0 or won[-1] == final[w] - 1, (w, final[w])
                assert np.array_equal(won, np.arange(final[w] - won.size, final[w])), w
            assert (final > 0).all()
        assert s.status() == 0


@pytest.mark.parametrize("staged", [0, 1])
def test_pingpong_phase_breakdown_moves_the_data_and_adds_up(staged):
    """The instrumented exchange: the payload arrives on both sides (bit-exact against the oracle's
    put_signal), both signal words count the rounds, and each side's five phases add up to its round
    (two half round trips by the global timer, within the clocks' disagreement)."""
    with Session(2, 1 << 16) as s:
        data, sig = s.malloc(4096), s.malloc(64)
        n, rounds = 256, 500
        data.fill(0, inputs.byte_payload(inputs.SEED_C4, 7, n))
        ph = np.zeros(14)
        B.ishmemx_pingpong_phases(0, 1, data.addr, sig.addr, n, rounds, 64, staged, ph)
        assert s.status() == 0
        s.oracle.putmem_signal(0, data.ooff, s.oracle.ptr(data.ooff, n, 0), n, sig.ooff, rounds, orc.SIG_SET, 1)
        s.oracle.putmem_signal(1, data.ooff, s.oracle.ptr(data.ooff, n, 1), n, sig.ooff, rounds, orc.SIG_SET, 0)
        heaps_equal(s, "instrumented ping-pong")
        assert (ph[:10] >= 0).all() and ph[10] > 50 and ph[11] > ph[12] > 0 and ph[13] > 0
        for side in (0, 1):
            assert abs(ph[5 * side:5 * side + 5].sum() - 2 * ph[13]) < 0.25 * 2 * ph[13], (side, ph)
        with pytest.raises(B.IshmemError):
            B.ishmemx_pingpong_phases(0, 0, data.addr, sig.addr, n, rounds, 64, staged, ph)
