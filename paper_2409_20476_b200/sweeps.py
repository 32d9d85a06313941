"""Message-size sweeps of the library on one B200, one sub-command per benchmark configuration.

    python -m paper_2409_20476_b200.sweeps --config 2 --out sweep_c2.csv

Timing follows the method of the paper's Section 4: the iteration count is doubled until
one batch of back-to-back operations lasts longer than 2 ms, then 10 batches are timed and
the best is kept.  Host-launched operations are timed with CUDA events on the stream they
are launched on; the in-kernel latencies come from ``ishmemx_rma_latency`` and
``ishmemx_pingpong`` (device global timer).  Bandwidth is *algorithmic* bytes (read plus
written, summed over the PEs that run concurrently) over time; ``frac_hbm`` divides by the
measured copy peak given with ``--peak-gbs`` and ``frac_8tbs`` by the nominal 8 TB/s.

``l2 = hot`` rows reuse one pair of buffers, so everything up to a few MiB per PE is served
by the 126 MB L2 and can exceed the HBM line; ``l2 = cold`` rows rotate through the whole
256 MiB buffers so that consecutive operations touch memory that has left L2.
"""
from __future__ import annotations

import argparse
import csv
import sys
from pathlib import Path

import numpy as np

MiB = 1 << 20
FIELDS = ["config", "op", "pattern", "variant", "level", "threads", "groups", "npes", "dtype", "nbytes",
          "l2", "iters", "us_per_op", "gbps", "frac_hbm", "frac_8tbs", "mops", "note"]


class Timer:
    def __init__(self, torch, stream, min_ms=2.0, trials=10, max_iters=1 << 13):
        self.torch, self.stream = torch, stream
        self.min_ms, self.trials, self.max_iters = min_ms, trials, max_iters

    def batch(self, fn, iters) -> float:
        t = self.torch
        a, b = t.cuda.Event(enable_timing=True), t.cuda.Event(enable_timing=True)
        t.cuda.synchronize()
        a.record(self.stream)
        for i in range(iters):
            fn(i)
        b.record(self.stream)
        t.cuda.synchronize()
        return a.elapsed_time(b)

    def __call__(self, fn):
        """-> (microseconds per call, iterations per batch)."""
        iters = 1
        self.batch(fn, 1)
        while True:
            ms = self.batch(fn, iters)
            if ms >= self.min_ms or iters >= self.max_iters:
                break
            iters *= 2
        trials = self.trials if ms < 50 else 3
        best = min([ms] + [self.batch(fn, iters) for _ in range(trials)])
        return best / iters * 1e3, iters


class Out:
    def __init__(self, path, peak_gbs):
        self.rows, self.path, self.peak = [], path, peak_gbs

    def add(self, **kw):
        us, nb = kw.get("us_per_op"), kw.pop("alg_bytes", None)
        if nb is not None and us:
            g = nb / us / 1e3
            kw["gbps"] = round(g, 2)
            kw["frac_hbm"] = round(g / self.peak, 4)
            kw["frac_8tbs"] = round(g / 8000.0, 4)
        if us is not None:
            kw["us_per_op"] = round(us, 3)
        self.rows.append({k: kw.get(k, "") for k in FIELDS})
        r = self.rows[-1]
        print(",".join(str(r[k]) for k in FIELDS), file=sys.stderr, flush=True)

    def write(self):
        Path(self.path).parent.mkdir(parents=True, exist_ok=True)
        with open(self.path, "w", newline="") as f:
            w = csv.DictWriter(f, fieldnames=FIELDS)
            w.writeheader()
            w.writerows(self.rows)


def _session(torch, B, npes, heap_bytes):
    heap = torch.empty(npes * heap_bytes, dtype=torch.uint8, device="cuda")
    B.ishmemx_init_external(npes, heap_bytes, heap.data_ptr())
    stream = torch.cuda.Stream()
    B.ishmemx_set_stream(-1, stream.cuda_stream)
    return heap, stream


def _fill_bytes(torch, heap, npes, heap_bytes, off, nbytes, seed, inputs):
    """uniform random bytes, one seeded 16 MiB block per PE tiled over [off, off+nbytes)"""
    for p in range(npes):
        blk = torch.from_numpy(inputs.byte_payload(seed, p, min(nbytes, 16 * MiB))).cuda()
        view = heap[p * heap_bytes + off:p * heap_bytes + off + nbytes]
        if nbytes > blk.numel():
            view.view(-1, blk.numel())[:] = blk
        else:
            view.copy_(blk)


# ------------------------------------------------------------------------------ config 2 ---

def sweep_c2(args, out):
    """8 PEs x 512 MiB: put/get, 8 B..256 MiB, every collaboration level and the copy engine,
    ring and all-pairs, plus the host API's adaptive path on one PE."""
    import torch
    from . import binding as B
    from . import inputs

    npes, heap_bytes, big = 8, 512 * MiB, 256 * MiB
    heap, stream = _session(torch, B, npes, heap_bytes)
    src, dst = B.ishmem_malloc(big), B.ishmem_malloc(big)
    _fill_bytes(torch, heap, npes, heap_bytes, src - heap.data_ptr(), big, inputs.SEED_C2, inputs)
    T = Timer(torch, stream)
    T1 = Timer(torch, stream, max_iters=1)
    sizes = inputs.message_sizes(3, 28)
    if args.quick:
        sizes = sizes[::5]
    WI, SG, WG, BK = B.ISHMEMX_WORK_ITEM, B.ISHMEMX_SUB_GROUP, B.ISHMEMX_WORK_GROUP, B.ISHMEMX_WORK_GROUP_BULK
    variants = [("work_item", WI, 1, 1, 4 * MiB), ("sub_group", SG, 32, 1, 64 * MiB)]
    variants += [(f"work_group_{t}x1", WG, t, 1, big) for t in (16, 128, 256, 1024)]
    variants += [(f"work_group_256x{g}", WG, 256, g, big) for g in (4, 18, 37, 74)]
    variants += [(f"work_group_512x{g}", WG, 512, g, big) for g in (37, 74)]
    variants += [(f"work_group_bulk_256x{g}", BK, 256, g, big) for g in (1, 4, 18, 37)]
    # groups = 0: the library sizes the grid, one tile of threads x 128 bytes per block
    variants += [("work_group_tiled_256", WG, 256, 0, big)]
    # device-initiated copy engine: each work-group's leader posts its slice to the host proxy
    B.ishmemx_proxy_start()
    B.ishmemx_set_wait_limit_ns(200_000_000)      # a lost reply costs 0.2 s, not 2 s, and shows in the status
    EN = B.ISHMEMX_WORK_GROUP_ENGINE
    variants += [(f"work_group_engine_{t}x{g}", EN, t, g, big) for t, g in ((64, 1), (1024, 1), (64, 4))]

    def slots(n):
        stride = max((n + 255) // 256 * 256, big // 1024)
        return max(1, big // stride), stride

    for op in ("put", "get"):
        spmd = B.ishmemx_putmem_spmd if op == "put" else B.ishmemx_getmem_spmd
        for name, level, threads, groups, cap in variants:
            for n in sizes:
                if n > cap:
                    continue
                # a kernel that waits for the host proxy must not have later launches queued behind
                # it (they can sit in front of the proxy's copy in a shared hardware queue): the
                # engine variants are timed one launch per batch
                timer = T1 if level == EN else T
                us, it = timer(lambda i: spmd(dst, src, n, 1, level, threads, groups))
                out.add(config=2, op=op, pattern="ring", variant=name, level=level, threads=threads, groups=groups,
                        npes=npes, dtype="u8", nbytes=n, l2="hot", iters=it, us_per_op=us, alg_bytes=2 * n * npes)
                if (groups >= 18 or groups == 0) and n < big:
                    nsl, stride = slots(n)
                    us, it = T(lambda i: spmd(dst + (i % nsl) * stride, src + (i % nsl) * stride, n, 1, level,
                                              threads, groups))
                    out.add(config=2, op=op, pattern="ring", variant=name, level=level, threads=threads,
                            groups=groups, npes=npes, dtype="u8", nbytes=n, l2="cold", iters=it, us_per_op=us,
                            alg_bytes=2 * n * npes)
    # copy engine, same pattern (8 cudaMemcpyAsync per operation)
    for n in sizes:
        us, it = T(lambda i: B.ishmemx_putmem_spmd_copy_engine(dst, src, n, 1))
        out.add(config=2, op="put", pattern="ring", variant="copy_engine", npes=npes, dtype="u8", nbytes=n, l2="hot",
                iters=it, us_per_op=us, alg_bytes=2 * n * npes)
        if n < big:
            nsl, stride = slots(n)
            us, it = T(lambda i: B.ishmemx_putmem_spmd_copy_engine(dst + (i % nsl) * stride, src + (i % nsl) * stride,
                                                                  n, 1))
            out.add(config=2, op="put", pattern="ring", variant="copy_engine", npes=npes, dtype="u8", nbytes=n,
                    l2="cold", iters=it, us_per_op=us, alg_bytes=2 * n * npes)
    # all-pairs: 7 permutation rounds p -> (p+r) mod 8 per operation
    for name, level, threads, groups in (("work_group_tiled_256", WG, 256, 0), ("work_group_bulk_256x37", BK, 256, 37),
                                          ("work_group_512x74", WG, 512, 74), ("copy_engine", None, 0, 0)):
        for n in sizes:
            def rounds(i, n=n):
                for r in range(1, npes):
                    if level is None:
                        B.ishmemx_putmem_spmd_copy_engine(dst, src, n, r)
                    else:
                        B.ishmemx_putmem_spmd(dst, src, n, r, level, threads, groups)
            us, it = T(rounds)
            out.add(config=2, op="put", pattern="all_pairs", variant=name, level=level if level is not None else "",
                    threads=threads, groups=groups, npes=npes, dtype="u8", nbytes=n, l2="hot", iters=it,
                    us_per_op=us / (npes - 1), alg_bytes=2 * n * npes, note="mean of the 7 rounds")
    # host API on ONE PE (PE 0 -> PE 1): the load/store kernel against the copy engine -- the cutover
    s0 = torch.cuda.Stream()
    B.ishmemx_set_stream(0, s0.cuda_stream)
    T0 = Timer(torch, s0)
    B.ishmemx_set_cutover(5, B.SIZE_MAX)          # no upper end: cutover 0 alone selects the path
    for n in sizes:
        B.ishmemx_set_cutover(0, B.SIZE_MAX)
        us, it = T0(lambda i: B.ishmem_putmem(0, dst, src, n, 1))
        out.add(config=2, op="put", pattern="one_pe", variant="host_api_kernel", npes=1, dtype="u8", nbytes=n,
                l2="hot", iters=it, us_per_op=us, alg_bytes=2 * n)
        B.ishmemx_set_cutover(0, 0)
        us, it = T0(lambda i: B.ishmem_putmem(0, dst, src, n, 1))
        out.add(config=2, op="put", pattern="one_pe", variant="host_api_copy_engine", npes=1, dtype="u8", nbytes=n,
                l2="hot", iters=it, us_per_op=us, alg_bytes=2 * n)
    B.ishmemx_set_cutover(0, B.SIZE_MAX)
    # strided put (iput) of one PE, PE 0 -> PE 1: element size, the two strides, element count
    span = 256 * MiB
    for es in (4, 8, 16):
        for dstride, sstride in ((1, 1), (2, 1), (1, 2), (2, 2), (4, 4), (8, 8), (64, 64)):
            for k in range(10, 26, 2):
                ne = 1 << k
                if ne * max(dstride, sstride) * es > span:
                    continue
                us, it = T0(lambda i: B.ishmemx_iputmem(0, dst, src, dstride, sstride, ne, es, 1))
                touched = ne * (min(32, dstride * es) + min(32, sstride * es))
                out.add(config=2, op="iput", pattern="strided", variant=f"es{es}_dst{dstride}_sst{sstride}", level=es,
                        threads=dstride, groups=sstride, npes=1, dtype="u8", nbytes=ne * es, l2="hot" if ne * es * max(dstride, sstride) < 32 * MiB else "cold",
                        iters=it, us_per_op=us, alg_bytes=2 * ne * es,
                        note=f"level = element size, threads = dest stride, groups = source stride (elements); "
                             f"sectors touched carry {touched} bytes")
    # device-timed latency of one collaboration unit (in-kernel loop, PE 0 -> PE 1)
    ns = np.zeros(1)
    for op, is_get in (("put", 0), ("get", 1)):
        for name, level, threads, cap in (("work_item", WI, 32, 1 * MiB), ("sub_group", SG, 32, 16 * MiB),
                                          ("work_group_16", WG, 16, 16 * MiB), ("work_group_128", WG, 128, 64 * MiB),
                                          ("work_group_256", WG, 256, 64 * MiB),
                                          ("work_group_1024", WG, 1024, 64 * MiB),
                                          ("work_group_bulk_256", BK, 256, 64 * MiB),
                                          ("work_group_engine_64", EN, 64, 64 * MiB)):
            for n in sizes:
                if n > cap:
                    continue
                iters = int(max(4, min(2000, (64 * MiB) // max(n, 4096))))
                B.ishmemx_rma_latency(0, dst, src, n, 1, is_get, level, threads, iters, ns)
                B.ishmemx_rma_latency(0, dst, src, n, 1, is_get, level, threads, iters, ns)
                out.add(config=2, op=op, pattern="one_pe", variant="in_kernel_" + name, level=level, threads=threads,
                        groups=1, npes=1, dtype="u8", nbytes=n, l2="hot", iters=iters, us_per_op=float(ns[0]) / 1e3,
                        alg_bytes=2 * n, note="device global timer, op + quiet")
    # hybrid put: above the cutover the engine takes the tail while the group copies the head
    B.ishmemx_set_cutover(3, 256 << 10)
    for head in (512 << 10, 1 * MiB, 2 * MiB):
        B.ishmemx_set_cutover(4, head)
        for n in sizes:
            if n < MiB or n > 64 * MiB:
                continue
            iters = int(max(4, min(200, (64 * MiB) // n)))
            B.ishmemx_rma_latency(0, dst, src, n, 1, 0, WG, 1024, iters, ns)
            B.ishmemx_rma_latency(0, dst, src, n, 1, 0, WG, 1024, iters, ns)
            out.add(config=2, op="put", pattern="one_pe", variant=f"in_kernel_hybrid_1024_head_{head >> 10}K", level=WG,
                    threads=1024, groups=1, npes=1, dtype="u8", nbytes=n, l2="hot", iters=iters,
                    us_per_op=float(ns[0]) / 1e3, alg_bytes=2 * n, note="device global timer, op + quiet")
    B.ishmemx_set_cutover(4, 0)
    B.ishmemx_set_cutover(3, B.SIZE_MAX)
    assert B.ishmemx_status(1) == 0
    B.ishmemx_proxy_stop()
    B.ishmem_finalize()


# ----------------------------------------------------------------- reverse-offload ring ---

def sweep_ring(args, out):
    """GPU -> host -> GPU round trip and request rate of the reverse-offload ring (64-byte
    requests, one host proxy thread), for growing numbers of posting GPU threads."""
    import torch
    from . import binding as B

    heap, stream = _session(torch, B, 2, 1 << 20)
    B.ishmemx_proxy_start()
    rtt, rate = np.zeros(1), np.zeros(1)
    memops = np.zeros(1, np.int32)
    B.ishmemx_proxy_stats(None, None, memops)
    for blocks, threads in ((1, 1), (1, 32), (1, 256), (8, 256), (32, 128), (148, 32), (148, 256)):
        iters = 400 if blocks * threads <= 256 else 100
        B.ishmemx_ring_benchmark(0, blocks, threads, iters, rtt, None)
        B.ishmemx_ring_benchmark(0, blocks, threads, iters, rtt, rate)
        out.add(config=6, op="ring_round_trip", pattern="gpu->host->gpu", variant="reply_per_request", threads=threads,
                groups=blocks, nbytes=64, iters=iters, us_per_op=float(rtt[0]) / 1e3, mops=round(float(rate[0]) / 1e6, 3),
                note=f"mean round trip per request; stream memory operations {'on' if memops[0] else 'off'}")
        B.ishmemx_ring_benchmark(1, blocks, threads, iters * 4, None, rate)
        B.ishmemx_ring_benchmark(1, blocks, threads, iters * 4, None, rate)
        out.add(config=6, op="ring_request_rate", pattern="gpu->host", variant="fire_and_forget", threads=threads,
                groups=blocks, nbytes=64, iters=iters * 4, us_per_op=1e6 / float(rate[0]),
                mops=round(float(rate[0]) / 1e6, 3), note="requests/s as seen from the GPU, one proxy thread")
    assert B.ishmemx_status(1) == 0
    B.ishmemx_proxy_stop()
    B.ishmem_finalize()


# ------------------------------------------------------------------------------ config 1 ---

def sweep_c1(args, out):
    """4 PEs x 16 MiB: work-group put/get of int32 messages 4 B..1 MiB on the ring, then the
    int32 sum_reduce of 262144 elements."""
    import torch
    from . import binding as B
    from . import inputs

    npes, heap_bytes = 4, 16 * MiB
    heap, stream = _session(torch, B, npes, heap_bytes)
    src, dst = B.ishmem_malloc(MiB), B.ishmem_malloc(MiB)
    for p in range(npes):
        v = torch.from_numpy(inputs.int32_payload(inputs.SEED_C1, p, MiB // 4)).cuda().view(torch.uint8)
        o = p * heap_bytes + src - heap.data_ptr()
        heap[o:o + MiB].copy_(v)
    T = Timer(torch, stream)
    ns = np.zeros(1)
    for n in inputs.message_sizes(2, 20):
        groups = max(1, min(37, n // 16384))
        for op, fn in (("put", B.ishmemx_putmem_spmd), ("get", B.ishmemx_getmem_spmd)):
            us, it = T(lambda i: fn(dst, src, n, 1, B.ISHMEMX_WORK_GROUP, 256, groups))
            out.add(config=1, op=op, pattern="ring", variant=f"work_group_256x{groups}", level=B.ISHMEMX_WORK_GROUP,
                    threads=256, groups=groups, npes=npes, dtype="i32", nbytes=n, l2="hot", iters=it, us_per_op=us,
                    alg_bytes=2 * n * npes, note="host-launched, all 4 PEs in one launch")
            iters = int(max(4, min(2000, (16 * MiB) // max(n, 4096))))
            B.ishmemx_rma_latency(0, dst, src, n, 1, int(op == "get"), B.ISHMEMX_WORK_GROUP, 256, iters, ns)
            out.add(config=1, op=op, pattern="one_pe", variant="in_kernel_work_group_256", level=B.ISHMEMX_WORK_GROUP,
                    threads=256, groups=1, npes=1, dtype="i32", nbytes=n, l2="hot", iters=iters,
                    us_per_op=float(ns[0]) / 1e3, alg_bytes=2 * n, note="device global timer, op + quiet")
    n = 262144
    for p in range(npes):
        v = torch.from_numpy(inputs.int32_reduce_values(inputs.SEED_C1, p, n)).cuda().view(torch.uint8)
        o = p * heap_bytes + src - heap.data_ptr()
        heap[o:o + 4 * n].copy_(v)
    for alg, name in ((B.ISHMEMX_REDUCE_SPLIT, "split"), (B.ISHMEMX_REDUCE_DUPLICATED, "duplicated")):
        us, it = T(lambda i: B.ishmemx_reduce(B.ISHMEM_TEAM_WORLD, dst, src, n, B.ISHMEM_OP_SUM, B.ISHMEM_T_INT32, alg))
        out.add(config=1, op="sum_reduce", pattern="team", variant=name, npes=npes, dtype="i32", nbytes=4 * n,
                l2="hot", iters=it, us_per_op=us, alg_bytes=2 * npes * 4 * n)
    assert B.ishmemx_status(1) == 0
    B.ishmem_finalize()


# ------------------------------------------------------------------------------ config 3 ---

def sweep_c3(args, out):
    """12 PEs: sum/max/min/prod reduce on float32, float64, int64; broadcast from root 0;
    fcollect; 1..64 Mi elements in powers of 4; stores against the copy engine for the push
    collectives; device-resident forms (one work-group per PE, in-kernel sync) for small sizes."""
    import torch
    from . import binding as B
    from . import inputs

    npes = 12
    max_el = (4 ** 13) if not args.quick else (4 ** 11)
    fc_el = min(max_el, args.fcollect_max_elems)
    heap_bytes = 8 * max_el + 8 * fc_el * npes + 4 * MiB
    heap, stream = _session(torch, B, npes, heap_bytes)
    src = B.ishmem_malloc(8 * max_el)
    dst = B.ishmem_malloc(max(8 * max_el, 8 * fc_el * npes))
    T = Timer(torch, stream)
    W = B.ISHMEM_TEAM_WORLD
    counts = [4 ** k for k in range(0, 14) if 4 ** k <= max_el]
    types = [("f32", np.float32, B.ISHMEM_T_FLOAT, 4), ("f64", np.float64, B.ISHMEM_T_DOUBLE, 8),
             ("i64", np.int64, B.ISHMEM_T_INT64, 8)]
    ops = [("sum", B.ISHMEM_OP_SUM), ("max", B.ISHMEM_OP_MAX), ("min", B.ISHMEM_OP_MIN), ("prod", B.ISHMEM_OP_PROD)]
    blk_el = MiB
    for tname, npdt, dt, es in types:
        for p in range(npes):
            if tname == "i64":
                v = inputs.int64_values(inputs.SEED_C3, p, blk_el)
            else:
                v = inputs.normal_values(inputs.SEED_C3, p, blk_el, npdt)
            blk = torch.from_numpy(v).cuda().view(torch.uint8)
            o = p * heap_bytes + src - heap.data_ptr()
            heap[o:o + es * max_el].view(-1, blk.numel())[:] = blk
        for n in counts:
            for oname, op in ops:
                us, it = T(lambda i: B.ishmemx_reduce(W, dst, src, n, op, dt, B.ISHMEMX_REDUCE_AUTO))
                out.add(config=3, op=oname + "_reduce", pattern="team", variant="auto", npes=npes, dtype=tname,
                        nbytes=n * es, l2="hot", iters=it, us_per_op=us, alg_bytes=2 * npes * n * es)
            if n * es <= 4 * MiB:
                us, it = T(lambda i: B.ishmemx_reduce(W, dst, src, n, B.ISHMEM_OP_SUM, dt, B.ISHMEMX_REDUCE_DUPLICATED))
                out.add(config=3, op="sum_reduce", pattern="team", variant="duplicated", npes=npes, dtype=tname,
                        nbytes=n * es, l2="hot", iters=it, us_per_op=us, alg_bytes=2 * npes * n * es)
            B.ishmemx_set_cutover(1, B.SIZE_MAX)
            us, it = T(lambda i: B.ishmem_broadcastmem(W, dst, src, n * es, 0))
            out.add(config=3, op="broadcast", pattern="team", variant="stores", npes=npes, dtype=tname, nbytes=n * es,
                    l2="hot", iters=it, us_per_op=us, alg_bytes=n * es * (1 + npes))
            if n <= fc_el:
                B.ishmemx_set_cutover(2, B.SIZE_MAX)
                us, it = T(lambda i: B.ishmem_fcollectmem(W, dst, src, n * es))
                out.add(config=3, op="fcollect", pattern="team", variant="stores", npes=npes, dtype=tname,
                        nbytes=n * es, l2="hot", iters=it, us_per_op=us, alg_bytes=n * es * (npes + npes * npes))
    # push collectives: stores against the copy engine, team sizes 2..12 (bytes; type-agnostic)
    for P in (2, 4, 8, 12):
        team = W if P == npes else B.ishmem_team_split_strided(W, 0, 1, P)
        for n in [4 ** k for k in range(1, 14) if 4 ** k <= 4 * fc_el]:
            for which, opname, fn, nb in ((1, "broadcast", lambda i: B.ishmem_broadcastmem(team, dst, src, n, 0),
                                          n * (1 + P)),
                                         (2, "fcollect", lambda i: B.ishmem_fcollectmem(team, dst, src, n),
                                          n * (P + P * P))):
                for variant, cut in (("stores", B.SIZE_MAX), ("copy_engine", 0)):
                    B.ishmemx_set_cutover(which, cut)
                    us, it = T(fn)
                    out.add(config=3, op=opname, pattern="team", variant=variant, npes=P, dtype="u8", nbytes=n,
                            l2="hot", iters=it, us_per_op=us, alg_bytes=nb)
        B.ishmemx_set_cutover(1, B.SIZE_MAX)
        B.ishmemx_set_cutover(2, B.SIZE_MAX)
        for n in [4 ** k for k in range(1, 13) if 4 ** k * P <= 8 * max_el]:
            us, it = T(lambda i: B.ishmem_alltoallmem(team, dst, src, n))
            out.add(config=3, op="alltoall", pattern="team", variant="stores", npes=P, dtype="u8", nbytes=n, l2="hot",
                    iters=it, us_per_op=us, alg_bytes=2 * P * P * n, note="nbytes = one block; P*P blocks move")
        # device-resident forms: one work-group per PE, push sync inside the kernel, `rep` calls per launch
        rep = 50
        for threads in (128, 256, 1024):
            for n in [4 ** k for k in range(0, 12)]:
                for which, opname, nb in ((0, "broadcast", n * (1 + P)), (1, "fcollect", n * (P + P * P)),
                                          (2, "sum_reduce_f32", 2 * P * n)):
                    if which == 2 and n < 4:
                        continue
                    cnt = n // 4 if which == 2 else n
                    us, it = T(lambda i: B.ishmemx_collective_on_device(which, team, dst, src, cnt, 0, B.ISHMEM_OP_SUM,
                                                                       B.ISHMEM_T_FLOAT, threads, rep))
                    out.add(config=3, op=opname, pattern="team", variant="device_resident", threads=threads, groups=1,
                            npes=P, dtype="u8", nbytes=n, l2="hot", iters=it * rep, us_per_op=us / rep, alg_bytes=nb,
                            note="one work-group per PE, in-kernel push sync")
            us, it = T(lambda i: B.ishmemx_collective_on_device(3, team, None, None, 0, 0, 0, 0, threads, rep))
            out.add(config=3, op="sync", pattern="team", variant="device_resident", threads=threads, groups=1, npes=P,
                    dtype="", nbytes=0, l2="hot", iters=it * rep, us_per_op=us / rep)
        if team != W:
            B.ishmem_team_destroy(team)
    assert B.ishmemx_status(1) == 0
    B.ishmem_finalize()


# ------------------------------------------------------------------------------ config 4 ---

def sweep_c4(args, out):
    """16 PEs: 2^22 fetch_add on 4096 words (Zipf 1.1) and on a uniform index stream, 2^20
    compare_swap on 1024 words, put_signal / wait_until ping-pong 8 B..64 KiB."""
    import torch
    from . import binding as B
    from . import inputs

    npes, heap_bytes = 16, 4 * MiB
    heap, stream = _session(torch, B, npes, heap_bytes)
    table = B.ishmem_calloc(4096, 8)
    data, sig = B.ishmem_malloc(64 << 10), B.ishmem_calloc(8, 8)
    T = Timer(torch, stream)
    nops, nwords = 1 << 22, 4096
    inc = torch.from_numpy(inputs.increments(inputs.SEED_C4, 0, nops)).cuda()
    fetched = torch.empty(nops, dtype=torch.int64, device="cuda")
    streams = {"zipf1.1": inputs.zipf_indices(inputs.SEED_C4, 0, nops, nwords),
               "uniform": inputs.rng_for(inputs.SEED_C4, 42).integers(0, nwords, nops).astype(np.int32),
               "one_word": np.zeros(nops, dtype=np.int32)}
    for sname, idx in streams.items():
        word = torch.from_numpy(idx).cuda()
        for agg in (2, 1, 0):
            for fet, fname in ((fetched, "fetch_add"), (None, "add")):
                for threads in (256, 1024):
                    us, it = T(lambda i: B.ishmemx_int64_atomic_fetch_add_batch(table, word, inc, fet, nops, threads, agg))
                    out.add(config=4, op=fname, pattern=sname, variant=("plain", "aggregate_warp", "aggregate_block")[agg],
                            threads=threads, npes=npes, dtype="i64", nbytes=8, l2="hot", iters=it, us_per_op=us,
                            mops=round(nops / us, 1), note=f"{nops} ops on {nwords} words")
    nops_c, nwords_c = 1 << 20, 1024
    cword = torch.from_numpy(inputs.zipf_indices(inputs.SEED_C4, 1, nops_c, nwords_c)).cuda()
    cval = torch.arange(1, nops_c + 1, dtype=torch.int64, device="cuda")
    for cname, ccond in (("claim_cond_0", torch.zeros(nops_c, dtype=torch.int64, device="cuda")),
                         ("never_matches", torch.full((nops_c,), -7, dtype=torch.int64, device="cuda"))):
        for agg in (1, 0):
            us, it = T(lambda i: B.ishmemx_int64_atomic_compare_swap_batch(table, cword, ccond, cval, fetched, nops_c,
                                                                           256, agg))
            out.add(config=4, op="compare_swap", pattern="zipf1.1", variant=cname + ("_aggregate_warp" if agg else "_plain"),
                    threads=256, npes=npes, dtype="i64", nbytes=8, l2="hot", iters=it, us_per_op=us,
                    mops=round(nops_c / us, 1), note=f"{nops_c} ops on {nwords_c} words")
    rtt, bad = np.zeros(1), np.zeros(1, dtype=np.uint64)
    rounds = 1000
    for threads in (32, 256, 1024):
        for n in inputs.message_sizes(3, 16):
            for a, b in ((0, 1),):
                B.ishmem_uint64_p(a, sig, 0, a)
                B.ishmem_uint64_p(b, sig, 0, b)
                B.ishmemx_pingpong(a, b, data, sig, n, rounds, threads, rtt, bad)
                out.add(config=4, op="put_signal_pingpong", pattern="pe0<->pe1", variant="in_kernel", threads=threads,
                        groups=1, npes=2, dtype="u8", nbytes=n, l2="hot", iters=rounds, us_per_op=float(rtt[0]) / 1e3,
                        alg_bytes=2 * n + 8, note=f"half round trip; stamp mismatches {int(bad[0])}")
    # where a half round trip goes: the instrumented exchange, context in global memory and in shared memory
    ph = np.zeros(14)
    names = ("wait", "translate", "copy", "barrier", "release")
    for staged in (0, 1):
        for threads in (32, 256):
            for n in (8, 256, 4096):
                for rep in range(2):
                    B.ishmem_uint64_p(0, sig, 0, 0)
                    B.ishmem_uint64_p(1, sig, 0, 1)
                    B.ishmemx_pingpong_phases(0, 1, data, sig, n, 2000, threads, staged, ph)
                note = "; ".join(f"{side} " + " ".join(f"{nm} {ph[5 * k + i]:.0f}" for i, nm in enumerate(names))
                                 for k, side in enumerate("AB"))
                note += f"; L2 trip {ph[10]:.0f}; store+release {ph[11]:.0f}; release alone {ph[12]:.0f}"
                out.add(config=4, op="pingpong_phases", pattern="pe0<->pe1",
                        variant="context_in_shared_memory" if staged else "context_in_global_memory", threads=threads,
                        groups=1, npes=2, dtype="u8", nbytes=n, l2="hot", iters=2000, us_per_op=float(ph[13]) / 1e3,
                        note="ns per round: " + note)
    assert B.ishmemx_status(1) == 0
    B.ishmem_finalize()


# ------------------------------------------------------------------------------ config 5 ---

def sweep_c5(args, out):
    """12 PEs: float64 5-point Jacobi on 16384 x 16384, 200 sweeps, halo rows by in-kernel
    work-group put_signal; with and without the interior-first overlap."""
    import torch
    from . import binding as B
    from . import inputs

    npes, n, iters = 12, (16384 if not args.quick else 4096), 200
    rows_max = -(-n // npes)
    nbytes = (rows_max + 2) * n * 8
    heap_bytes = 2 * nbytes + 2 * MiB     # the buffers, the signals and the call's own halo rows
    heap, stream = _session(torch, B, npes, heap_bytes)
    b0, b1, sig = B.ishmem_malloc(nbytes), B.ishmem_malloc(nbytes), B.ishmem_calloc(4, 8)
    base, extra = divmod(n, npes)
    res = np.zeros(1)

    def load():
        first = 0
        heap.zero_()
        for p in range(npes):
            rows = base + (1 if p < extra else 0)
            win = inputs.jacobi_cell_init(inputs.SEED_C5, n, n, first, first + rows, 0, n)
            o = p * heap_bytes + (b0 - heap.data_ptr()) + n * 8
            heap[o:o + rows * n * 8].copy_(torch.from_numpy(win.view(np.uint8).ravel()))
            first += rows

    load()
    # (variant, form selected through ishmemx_set_option, threads, groups): the launch-ordered forms (the library's own
    # choice: six sweeps per launch; at most five, four, three, two, one), the persistent kernel with strips cut by
    # column tiles, and the persistent kernel with caller-shaped blocks
    variants = [("launch_per_six_sweeps", 1, 0, 1), ("launch_per_five_sweeps", 5, 0, 1), ("launch_per_four_sweeps", 4, 0, 1),
                ("launch_per_three_sweeps", 3, 0, 1), ("launch_per_two_sweeps", 2, 0, 1), ("launch_per_sweep", 0, 0, 1)]
    variants += [("persistent_columns", "columns", 0, g) for g in (6, 12)]
    variants += [("persistent_rows", "rows", t, g) for g in (6, 12, 24) for t in (256, 512, 1024)]
    if args.quick:
        variants = variants[:7]
    for overlap in (1, 0):
        for variant, split, threads, groups in variants:
            if npes * groups * threads > 148 * 2048:
                continue
            B.ishmemx_set_option(B.ISHMEMX_OPT_JACOBI_SPLIT, {"rows": 1, "columns": 2}.get(split, 0))
            B.ishmemx_set_option(B.ISHMEMX_OPT_JACOBI_FUSE, split if isinstance(split, int) else 1)
            # sweeps per launch of the bulk of the call (200 sweeps: 30 x 6 + 4 x 5, 40 x 5, 50 x 4, 66 x 3 + 1 + 1,
            # 100 x 2, 200 x 1)
            depth = {1: 6, 5: 5, 4: 4, 3: 3, 2: 2}.get(split, 1) if isinstance(split, int) else 1
            def reset_signals():
                for p in range(npes):
                    for w in range(4):
                        B.ishmem_uint64_p(p, sig + 8 * w, 0, p)
            try:
                # the same call untimed first: the first launch of a kernel in a process loads its code, and
                # the call launches kernels of several depths
                reset_signals()
                B.ishmemx_jacobi(b0, b1, sig, n, n, iters, overlap, groups, threads, res)
            except B.IshmemError:
                pass
            reset_signals()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record(stream)
            try:
                B.ishmemx_jacobi(b0, b1, sig, n, n, iters, overlap, groups, threads, res)
            except B.IshmemError as e:
                out.add(config=5, op="jacobi", variant=f"{variant} overlap={overlap}", threads=threads, groups=groups,
                        npes=npes, dtype="f64", nbytes=n * n * 8, note=str(e))
                continue
            b.record(stream)
            torch.cuda.synchronize()
            us = a.elapsed_time(b) * 1e3 / iters
            out.add(config=5, op="jacobi", pattern=f"{n}x{n}", variant=f"{variant} overlap={overlap}", level=depth,
                    threads=threads, groups=groups, npes=npes, dtype="f64", nbytes=n * n * 8, l2="cold", iters=iters,
                    us_per_op=us, alg_bytes=16 * n * n,
                    note=f"per sweep; level = sweeps per launch; residual_sq {res[0]:.6e} (grid keeps evolving)")
    # smaller square grids in the same buffers (timing only: the cells keep whatever the runs above left): the
    # library's own choice against a cap of four sweeps per launch and single sweeps
    B.ishmemx_set_option(B.ISHMEMX_OPT_JACOBI_SPLIT, 0)
    for m in ([512, 1024, 2048, 4096, 8192] if not args.quick else [512, 2048]):
        for variant, fuse in (("library_choice", 1), ("at_most_four_sweeps_per_launch", 4), ("launch_per_sweep", 0)):
            B.ishmemx_set_option(B.ISHMEMX_OPT_JACOBI_FUSE, fuse)
            best = None
            for rep in range(4):                     # the first call loads the kernels
                for p in range(npes):
                    for w in range(4):
                        B.ishmem_uint64_p(p, sig + 8 * w, 0, p)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                a.record(stream)
                B.ishmemx_jacobi(b0, b1, sig, m, m, 120, 1, 1, 0, None)
                b.record(stream)
                torch.cuda.synchronize()
                if rep:
                    best = min(best or 1e30, a.elapsed_time(b) * 1e3 / 120)
            out.add(config=5, op="jacobi_sizes", pattern=f"{m}x{m}", variant=variant, npes=npes, dtype="f64",
                    nbytes=m * m * 8, l2="resident" if 2 * m * m * 8 < 100 * MiB else "cold", iters=120, us_per_op=best,
                    alg_bytes=16 * m * m, note="per sweep, 120 sweeps per call, best of 3 calls")
    assert B.ishmemx_status(1) == 0
    B.ishmem_finalize()


# ------------------------------------------------------------------------------ summaries ---

def _fmt_size(n):
    n = int(n)
    for unit, k in (("GiB", 1 << 30), ("MiB", 1 << 20), ("KiB", 1 << 10)):
        if n >= k and n % k == 0:
            return f"{n // k} {unit}"
    return f"{n} B"


def _table(rows, row_key, col_key, val, row_fmt=str, cols=None):
    """markdown pivot: one line per row_key value, one column per col_key value"""
    cols = cols or list(dict.fromkeys(col_key(r) for r in rows))
    keys = list(dict.fromkeys(row_key(r) for r in rows))
    cell = {(row_key(r), col_key(r)): val(r) for r in rows}
    out = ["| size | " + " | ".join(cols) + " |", "|---:|" + "---:|" * len(cols)]
    for k in keys:
        out.append(f"| {row_fmt(k)} | " + " | ".join(str(cell.get((k, c), "")) for c in cols) + " |")
    return "\n".join(out)


def _crossover(a, b):
    """smallest size from which b's time is <= a's at every larger common size, or None"""
    pick = None
    for n in sorted(set(a) & set(b)):
        if b[n] <= a[n]:
            pick = n if pick is None else pick
        else:
            pick = None
    return pick


def _band(a, b):
    """longest run of consecutive common sizes at which b's time is <= a's: (first size of the
    run, first size after it at which a wins or None when the run reaches the top), or None"""
    best, run = None, []
    sizes = sorted(set(a) & set(b))
    for k, n in enumerate(sizes):
        if b[n] <= a[n]:
            run.append(n)
            if best is None or len(run) > best[2]:
                best = (run[0], sizes[k + 1] if k + 1 < len(sizes) else None, len(run))
        else:
            run = []
    if best is None:
        return None
    lo, after, _ = best
    return lo, (after if after is not None and b[after] > a[after] else None)


def summarize(path) -> str:
    rows = list(csv.DictReader(open(path)))
    cfg = int(rows[0]["config"])
    nb = lambda r: int(r["nbytes"])
    gb = lambda r: f"{float(r['gbps']):.0f}" if r["gbps"] else ""
    us = lambda r: f"{float(r['us_per_op']):.2f}" if r["us_per_op"] else ""
    out = []
    if cfg == 2:
        ring = [r for r in rows if r["pattern"] == "ring" and r["op"] == "put"]
        keep = ["work_item", "sub_group", "work_group_16x1", "work_group_128x1", "work_group_1024x1",
                "work_group_256x18", "work_group_512x74", "work_group_bulk_256x37", "work_group_tiled_256",
                "work_group_engine_64x1", "copy_engine"]
        for l2 in ("hot", "cold"):
            sel = [r for r in ring if r["l2"] == l2 and r["variant"] in keep]
            out += [f"### put, ring p -> (p+1) mod 8, 8 PEs concurrently, {l2} buffers: GB/s (algorithmic, aggregate)", "",
                    _table(sel, nb, lambda r: r["variant"], gb, _fmt_size, [k for k in keep if any(r["variant"] == k for r in sel)]), ""]
        t = lambda var, l2="hot", op="put", pat="ring": {nb(r): float(r["us_per_op"]) for r in rows if r["variant"] == var
                                                          and r["l2"] == l2 and r["op"] == op and r["pattern"] == pat}
        out += ["### crossover: smallest message from which the copy engine is at least as fast at every larger size", ""]
        for var in ("work_item", "sub_group", "work_group_16x1", "work_group_128x1", "work_group_256x1", "work_group_1024x1",
                    "work_group_256x4", "work_group_256x18", "work_group_256x37", "work_group_512x74",
                    "work_group_bulk_256x37", "work_group_tiled_256"):
            c = _crossover(t(var), t("copy_engine"))
            out.append(f"- `{var}` vs host-started copy engine (ring, 8 PEs): " + (_fmt_size(c) if c else "never"))
        band = _band(t("host_api_kernel", pat="one_pe"), t("host_api_copy_engine", pat="one_pe"))
        out.append("- host API `ishmem_putmem`, one PE, kernel vs engine: the engine is at least as fast from "
                   + (f"{_fmt_size(band[0])} up to " + (f"(not including) {_fmt_size(band[1])}" if band[1] else "the largest size")
                      if band else "no size")
                   + " -- a band, not a threshold (table below; defaults of cutover 0 and 5)")
        for var in ("in_kernel_work_item", "in_kernel_sub_group", "in_kernel_work_group_16", "in_kernel_work_group_128",
                    "in_kernel_work_group_256", "in_kernel_work_group_1024", "in_kernel_work_group_bulk_256"):
            c = _crossover(t(var, pat="one_pe"), t("in_kernel_work_group_engine_64", pat="one_pe"))
            out.append(f"- one collaboration unit inside a kernel, `{var[10:]}` vs device-initiated engine request: "
                       + (_fmt_size(c) if c else "never"))
        sel = [r for r in rows if r["pattern"] == "one_pe" and r["op"] == "put" and r["variant"].startswith("in_kernel")]
        out += ["", "### one collaboration unit, PE 0 -> PE 1, put + quiet timed inside the kernel: microseconds", "",
                _table(sel, nb, lambda r: r["variant"][10:], us, _fmt_size), ""]
        sel = [r for r in rows if r["pattern"] == "strided"]
        if sel:
            out += ["### strided put `ishmemx_iputmem`, one PE (PE 0 -> PE 1): GB/s of useful bytes (2 x elements x element size) / "
                    "GB/s of the bytes in the 32-byte sectors it has to touch", "",
                    "Column: element size, destination stride, source stride (in elements).  A stride of s elements of e bytes "
                    "touches min(32, s e) bytes per element on that side, so the second figure is what the memory system "
                    "moves; it is the one to hold against the copy rate.", ""]

            def both(r):
                touched = float(r["note"].rsplit("carry ", 1)[1].split()[0])
                t = float(r["us_per_op"])
                return f"{float(r['gbps']):.0f} / {touched / t / 1e3:.0f}"
            for es in ("4", "8", "16"):
                part = [r for r in sel if r["level"] == es]
                out += [f"elements of {es} bytes (row: number of elements; column: destination stride, source stride):", "",
                        _table(part, lambda r: nb(r) // int(es), lambda r: r["variant"].split("_", 1)[1].replace("_", " "), both,
                               lambda n: f"2^{int(n).bit_length() - 1}"), ""]
        sel = [r for r in rows if r["pattern"] == "one_pe" and r["variant"].startswith("host_api")]
        out += ["### host API `ishmem_putmem` on ONE PE (PE 0 -> PE 1), back-to-back calls: microseconds per call / GB/s", "",
                _table(sel, nb, lambda r: r["variant"][9:], lambda r: f"{us(r)} / {gb(r)}", _fmt_size), ""]
        sel = [r for r in rows if r["pattern"] == "all_pairs"]
        out += ["### all-pairs (mean of the 7 permutation rounds): GB/s", "",
                _table(sel, nb, lambda r: r["variant"], gb, _fmt_size), ""]
        getr = [r for r in rows if r["pattern"] == "ring" and r["op"] == "get" and r["l2"] == "hot"
                and r["variant"] in ("work_group_512x74", "work_group_bulk_256x37", "work_group_tiled_256")
                and nb(r) >= 1 << 20]
        out += ["### get, ring, hot buffers: GB/s", "", _table(getr, nb, lambda r: r["variant"], gb, _fmt_size), ""]
    elif cfg == 1:
        out += ["### 4 PEs x 16 MiB, int32: microseconds per operation", "",
                _table([r for r in rows if r["op"] in ("put", "get")], nb,
                       lambda r: r["op"] + " " + ("in-kernel" if r["variant"].startswith("in_kernel") else "host-launched x4 PEs"),
                       us, _fmt_size), ""]
        for r in rows:
            if r["op"] == "sum_reduce":
                out.append(f"- int32 sum_reduce, 262144 elements, 4 PEs, {r['variant']}: {us(r)} us ({gb(r)} GB/s algorithmic)")
    elif cfg == 3:
        for dt in ("f32", "f64", "i64"):
            sel = [r for r in rows if r["dtype"] == dt and r["variant"] in ("auto", "stores")]
            out += [f"### 12 PEs, {dt}: GB/s (algorithmic) / microseconds", "",
                    _table(sel, nb, lambda r: r["op"], lambda r: f"{gb(r)} / {us(r)}", _fmt_size), ""]
        for op in ("broadcast", "fcollect"):
            out += [f"### {op}: stores vs copy engine, microseconds", ""]
            sel = [r for r in rows if r["op"] == op and r["dtype"] == "u8" and r["variant"] in ("stores", "copy_engine")]
            out += [_table(sel, nb, lambda r: f"P={r['npes']} {r['variant']}", us, _fmt_size), ""]
            for P in ("2", "4", "8", "12"):
                a = {nb(r): float(r["us_per_op"]) for r in sel if r["npes"] == P and r["variant"] == "stores"}
                b = {nb(r): float(r["us_per_op"]) for r in sel if r["npes"] == P and r["variant"] == "copy_engine"}
                c = _crossover(a, b)
                out.append(f"- {op}, {P} PEs: engine at least as fast from " + (_fmt_size(c) if c else "never"))
            out.append("")
        sel = [r for r in rows if r["op"] == "alltoall"]
        if sel:
            out += ["### alltoall (block size per pair; P x P blocks move): GB/s (algorithmic 2 P^2 n) / microseconds", "",
                    _table(sel, nb, lambda r: f"P={r['npes']}", lambda r: f"{gb(r)} / {us(r)}", _fmt_size), ""]
        dev = [r for r in rows if r["variant"] == "device_resident"]
        for op in ("broadcast", "fcollect", "sum_reduce_f32", "sync"):
            sel = [r for r in dev if r["op"] == op]
            if not sel:
                continue
            out += [f"### device-resident {op} (one work-group of T work-items per PE, in-kernel push sync): microseconds", "",
                    _table(sel, nb, lambda r: f"P={r['npes']} T={r['threads']}", us, _fmt_size), ""]
            if op in ("broadcast", "fcollect"):
                eng = [r for r in rows if r["op"] == op and r["dtype"] == "u8" and r["variant"] == "copy_engine"]
                for P in ("2", "4", "8", "12"):
                    b = {nb(r): float(r["us_per_op"]) for r in eng if r["npes"] == P}
                    for T_ in ("128", "256", "1024"):
                        a = {nb(r): float(r["us_per_op"]) for r in sel if r["npes"] == P and r["threads"] == T_}
                        c = _crossover(a, b)
                        out.append(f"- {op}, {P} PEs, one work-group of {T_} work-items per PE against the host-started copy "
                                   f"engine: engine at least as fast from " + (_fmt_size(c) if c else "no size measured (<= 4 MiB)"))
                out.append("")
    elif cfg == 4:
        out += ["### remote atomics, 16 PEs: Mops/s (one op per GPU thread)", "", "| op | index stream | variant | threads | Mops/s | us |",
                "|---|---|---|---:|---:|---:|"]
        for r in rows:
            if r["mops"]:
                out.append(f"| {r['op']} | {r['pattern']} | {r['variant']} | {r['threads']} | {float(r['mops']):.0f} | {us(r)} |")
        sel = [r for r in rows if r["op"] == "pingpong_phases"]
        if sel:
            out += ["", "### where a half round trip goes (`ishmemx_pingpong_phases`): nanoseconds per round and side", "",
                    "Each side's five phases add up to its round (= two half round trips); `wait` on a side contains the other "
                    "side's translate + copy + barrier + release.  Cycle counter of the SM, converted at the nominal clock.", "",
                    "| context | threads | size | half rtt us | A: wait / translate / copy / barrier / release | "
                    "B: wait / translate / copy / barrier / release | L2 trip | store + release | release alone |",
                    "|---|---:|---:|---:|---|---|---:|---:|---:|"]
            for r in sel:
                f = r["note"].replace("ns per round: ", "").split("; ")
                side = lambda t: " / ".join(t.split()[2::2])
                out.append(f"| {r['variant'][11:].replace('_', ' ')} | {r['threads']} | {_fmt_size(r['nbytes'])} | {us(r)} | {side(f[0])} | "
                           f"{side(f[1])} | {f[2].split()[-1]} | {f[3].split()[-1]} | {f[4].split()[-1]} |")
        sel = [r for r in rows if r["op"] == "put_signal_pingpong"]
        out += ["", "### put_signal / wait_until ping-pong, half round trip in microseconds (in-kernel)", "",
                _table(sel, nb, lambda r: f"{r['threads']} threads", us, _fmt_size), ""]
    elif cfg == 5:
        out += ["### Jacobi 16384 x 16384 float64, 12 PEs, 200 sweeps: per sweep", "",
                "GB/s at 16 B per cell and sweep (the algorithmic figure of a single sweep); the last two columns count the "
                "bytes the form has to move -- 16 B per cell and LAUNCH, i.e. 16 / K per sweep -- against the measured copy rate.", "",
                "| form | overlap | threads | groups/PE | sweeps per launch K | us/sweep | us/launch | GB/s (16 B/cell/sweep) | "
                "of measured copy | of 8 TB/s | GB/s moved (16/K B) | of measured copy |",
                "|---|---|---:|---:|---:|---:|---:|---:|---:|---:|---:|---:|"]
        for r in [r for r in rows if r["op"] == "jacobi"]:
            form, ov = r["variant"].rsplit(" overlap=", 1) if " overlap=" in r["variant"] else ("", r["variant"][-1])
            k = int(r["level"] or 1)
            shape = (f"| {form} | {ov} | {r['threads'] if r['threads'] != '0' else 'library'} | "
                     f"{r['groups'] if not form.startswith('launch_per') else '-'} | {k} |")
            if r["us_per_op"]:
                moved = float(r["gbps"]) / k
                peak = float(r["gbps"]) / float(r["frac_hbm"])
                out.append(f"{shape} {us(r)} | {float(r['us_per_op']) * k:.1f} | {gb(r)} | {r['frac_hbm']} | {r['frac_8tbs']} | "
                           f"{moved:.0f} | {moved / peak:.3f} |")
            else:
                out.append(f"{shape} refused: not co-resident | | | | | | |")
        sel = [r for r in rows if r["op"] == "jacobi_sizes"]
        if sel:
            out += ["", "### Smaller square grids, 12 PEs, 120 sweeps per call: microseconds per sweep", "",
                    "Bands are lowered from 128 / 64 rows down to 16 until a launch has a dozen blocks per SM; the last column is one "
                    "pass over the grid (16 B per cell) at the measured copy rate, for scale -- grids up to 2048^2 stay in L2.", ""]
            peak = float(sel[0]["gbps"]) / float(sel[0]["frac_hbm"])
            tab = _table(sel, lambda r: r["pattern"], lambda r: r["variant"], us, str).splitlines()
            tab[0] = tab[0].replace("| size |", "| grid |") + " one pass at the copy rate |"
            tab[1] += "---:|"
            for i, m in enumerate(dict.fromkeys(r["pattern"] for r in sel)):
                n = int(m.split("x")[0])
                tab[2 + i] += f" {16.0 * n * n / peak / 1e3:.1f} |"
            out += tab
    elif cfg == 6:
        out += ["### reverse-offload ring (64-byte requests, one host proxy thread)", "",
                "| measurement | blocks x threads | us | M requests/s |", "|---|---:|---:|---:|"]
        for r in rows:
            out.append(f"| {r['op']} | {r['groups']} x {r['threads']} | {us(r)} | {r['mops']} |")
    return "\n".join(out) + "\n"


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--summarize", default=None, metavar="CSV", help="print a markdown digest of a CSV written earlier")
    ap.add_argument("--config", type=int, default=None, choices=[1, 2, 3, 4, 5, 6],
                    help="benchmark configuration 1..5, or 6 = the reverse-offload ring")
    ap.add_argument("--out", default=None, help="CSV file to write")
    ap.add_argument("--peak-gbs", type=float, default=None,
                    help="measured HBM copy peak in GB/s (default: MEASURED_PEAKS.json beside the package, else 6650)")
    ap.add_argument("--quick", action="store_true", help="fewer sizes (smoke run)")
    ap.add_argument("--fcollect-max-elems", type=int, default=4 ** 12,
                    help="largest per-PE element count of the 8-byte fcollect rows")
    args = ap.parse_args(argv)
    if args.summarize:
        print(summarize(args.summarize))
        return 0
    if args.config is None or args.out is None:
        ap.error("--config and --out are required")
    peak = args.peak_gbs
    if peak is None:
        import json
        f = Path(__file__).resolve().parent.parent / "MEASURED_PEAKS.json"
        peak = float(json.loads(f.read_text())["hbm_gbs"]) if f.exists() else 6650.0
    out = Out(args.out, peak)
    try:
        {1: sweep_c1, 2: sweep_c2, 3: sweep_c3, 4: sweep_c4, 5: sweep_c5, 6: sweep_ring}[args.config](args, out)
    finally:
        out.write()
    return 0


if __name__ == "__main__":
    sys.exit(main())
