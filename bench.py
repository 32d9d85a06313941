#!/usr/bin/env python
"""Benchmark of the GPU-initiated OpenSHMEM hot path on B200.

One *step* is one pass of the whole hot path over one batch of synthetic input on the
configuration the headline metric is quoted on: 8 logical PEs with a 512 MiB symmetric
heap each (4 GiB, far larger than L2, so no L2 flush is needed between steps):

  work-group put ring and get ring of 256 MiB per PE, work-item and sub-group puts, a
  scalar p, non-blocking puts through the copy engine + quiet, put_signal + wait_until,
  an in-kernel ping-pong, 2^22 fetch_add + 2^20 compare_swap remote atomics, broadcast,
  fcollect, float32 and int32 sum_reduce, a 4-sweep Jacobi with in-kernel halo put_signal,
  and barrier_all.

``value`` is the algorithmic bytes of a step (see ``step_bytes``) times the steps, over the
device time of the timed region, summed over ranks / max over ranks (replicas: nothing
spans a second GPU).  ``python bench.py --impl reference`` times the CPU oracle on a
bounded sample of the same step instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

MiB = 1 << 20
NPES = 8
HEAP = 512 * MiB
MSG = 256 * MiB          # put/get message per PE
NOPS_FADD, NWORDS_FADD = 1 << 22, 4096
NOPS_CAS, NWORDS_CAS = 1 << 20, 1024
JAC_N, JAC_SWEEPS = 4096, 4


def sizes(scale: int = 1) -> dict:
    """Per-op sizes of one step; scale > 1 shrinks them (the CPU sample)."""
    s = {
        "put": MSG // scale, "get": MSG // scale, "work_item": 64 << 10, "sub_group": MiB,
        "nbi": 64 * MiB // scale, "signal": 64 << 10, "pp_bytes": 4096, "pp_rounds": 100,
        "fadd_ops": NOPS_FADD // scale, "cas_ops": NOPS_CAS // scale,
        "bcast": 64 * MiB // scale, "fcollect": 16 * MiB // scale,
        "reduce_f32": 16 * MiB // scale, "reduce_i32": 262144,        # elements
        "jacobi_n": JAC_N if scale == 1 else max(256, int(JAC_N / scale ** 0.5) // 8 * 8),
        "jacobi_sweeps": JAC_SWEEPS,
    }
    return s


def step_bytes(s: dict, npes: int = NPES) -> dict:
    """Algorithmic bytes per op of one step (bytes that must be read plus written)."""
    P = npes
    return {
        "put": 2 * s["put"] * P, "get": 2 * s["get"] * P,
        "work_item": 2 * s["work_item"] * P, "sub_group": 2 * s["sub_group"] * P,
        "p": 8, "nbi": 2 * s["nbi"] * P, "signal": 2 * s["signal"] + 8,
        "pingpong": s["pp_rounds"] * 2 * (2 * s["pp_bytes"] + 8),
        "fetch_add": s["fadd_ops"] * (8 + 12 + 8), "compare_swap": s["cas_ops"] * (8 + 20 + 8),
        "broadcast": s["bcast"] * (1 + P), "fcollect": s["fcollect"] * (P + P * P),
        "reduce_f32": 2 * P * 4 * s["reduce_f32"], "reduce_i32": 2 * P * 4 * s["reduce_i32"],
        "jacobi": 16 * s["jacobi_n"] ** 2 * s["jacobi_sweeps"],
    }


# ------------------------------------------------------------------ clocks sampling ---

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.lines, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for nm, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm),
                "reasons": sorted(reasons)}


# ------------------------------------------------------------------------ GPU arm ---

def run_ours(args) -> dict:
    import torch
    from paper_2409_20476_b200 import binding as B
    from paper_2409_20476_b200 import inputs, replicas

    rank, local_rank, world = replicas.init()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    B.lib()  # fails loudly when libishmem.so has not been built

    heap = torch.empty(NPES * HEAP, dtype=torch.uint8, device="cuda")
    B.ishmemx_init_external(NPES, HEAP, heap.data_ptr())
    team_stream = torch.cuda.Stream()
    B.ishmemx_set_stream(-1, team_stream.cuda_stream)
    src = B.ishmem_malloc(MSG)
    dst = B.ishmem_malloc(MSG)
    assert src and dst
    S = sizes()
    nbytes = step_bytes(S)
    level = {"tiled": B.ISHMEMX_WORK_GROUP, "bulk": B.ISHMEMX_WORK_GROUP_BULK, "ldst": B.ISHMEMX_WORK_GROUP}[args.level]

    # seeded synthetic payload: uniform random bytes (config 2, seed 1), one block per PE
    for p in range(NPES):
        blk = torch.from_numpy(inputs.byte_payload(inputs.SEED_C2, p, 16 * MiB)).cuda()
        view = heap[p * HEAP:(p + 1) * HEAP]
        view[:MSG].view(-1, 16 * MiB)[:] = blk
        view[MSG:] = 0
        view[MSG - 256:MSG] = 0          # a zero source for resetting signal words (end of src)
    # the Jacobi strips live at the start of src: a proper float64 grid (config 5 recipe)
    jn = sizes()["jacobi_n"]
    grid = inputs.jacobi_grid(inputs.SEED_C5, jn, jn)
    rows = jn // NPES
    for p in range(NPES):
        strip = np.zeros((rows + 2, jn))
        strip[1:rows + 1] = grid[p * rows:(p + 1) * rows]
        heap[p * HEAP:p * HEAP + strip.nbytes].copy_(torch.from_numpy(strip.view(np.uint8).ravel()))
    word = torch.from_numpy(inputs.zipf_indices(inputs.SEED_C4, 0, NOPS_FADD, NWORDS_FADD)).cuda()
    inc = torch.from_numpy(inputs.increments(inputs.SEED_C4, 0, NOPS_FADD)).cuda()
    fetched = torch.empty(NOPS_FADD, dtype=torch.int64, device="cuda")
    cword = torch.from_numpy(inputs.zipf_indices(inputs.SEED_C4, 1, NOPS_CAS, NWORDS_CAS)).cuda()
    ccond = torch.zeros(NOPS_CAS, dtype=torch.int64, device="cuda")
    cval = torch.arange(1, NOPS_CAS + 1, dtype=torch.int64, device="cuda")
    # sub-ranges of dst used by the small ops (dst is rewritten by every step anyway)
    table, sig, ppdata, ppsig = dst, dst + 64 * 1024, dst + 128 * 1024, dst + 256 * 1024
    rows_max = -(-S["jacobi_n"] // NPES)
    jac_bytes = (rows_max + 2) * S["jacobi_n"] * 8
    jb0, jb1, jsig = src, dst + MiB, dst + 512 * 1024
    zeros = src + MSG - 256
    rtt, bad, res = np.zeros(1), np.zeros(1, dtype=np.uint64), np.zeros(1)
    ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731
    put_ev, get_ev = [], []
    step_no = [0]

    def step(record: bool):
        step_no[0] += 1
        k = step_no[0]
        if record:
            e0, e1, e2 = ev(), ev(), ev()
            e0.record(team_stream)
        B.ishmemx_putmem_spmd(dst, src, S["put"], 1, level, args.threads, args.groups)
        if record:
            e1.record(team_stream)
        B.ishmemx_getmem_spmd(dst, src, S["get"], 1, level, args.threads, args.groups)
        if record:
            e2.record(team_stream)
            put_ev.append((e0, e1))
            get_ev.append((e1, e2))
        B.ishmemx_putmem_spmd(dst, src, S["work_item"], 1, B.ISHMEMX_WORK_ITEM, 64, 1)
        B.ishmemx_putmem_spmd(dst, src, S["sub_group"], 2, B.ISHMEMX_SUB_GROUP, 256, 4)
        B.ishmem_long_p(0, dst, k, 1)
        B.ishmemx_set_cutover(0, 1 * MiB)              # from 1 MiB on, with no upper end: copy engine
        B.ishmemx_set_cutover(5, B.SIZE_MAX)
        for p in range(NPES):
            B.ishmem_putmem_nbi(p, dst, src, S["nbi"], (p + 1) % NPES)
        for p in range(NPES):
            B.ishmem_quiet(p)
        B.ishmemx_set_cutover(0, B.SIZE_MAX)
        B.ishmem_putmem_signal(0, dst + MiB, src, S["signal"], sig, k, B.ISHMEM_SIGNAL_SET, 1)
        B.ishmem_uint64_wait_until(1, sig, B.ISHMEM_CMP_GE, k)
        B.ishmem_uint64_p(0, ppsig, 0, 0)
        B.ishmem_uint64_p(1, ppsig, 0, 1)
        B.ishmemx_pingpong(0, 1, ppdata, ppsig, S["pp_bytes"], S["pp_rounds"], 256, rtt, bad)
        B.ishmemx_int64_atomic_fetch_add_batch(table, word, inc, fetched, NOPS_FADD, 1024, 2)
        B.ishmemx_int64_atomic_compare_swap_batch(table, cword, ccond, cval, fetched, NOPS_CAS, 256, 1)
        B.ishmem_broadcastmem(B.ISHMEM_TEAM_WORLD, dst, src, S["bcast"], 0)
        B.ishmem_fcollectmem(B.ISHMEM_TEAM_WORLD, dst, src, S["fcollect"])
        B.ishmem_float_sum_reduce(B.ISHMEM_TEAM_WORLD, dst, src, S["reduce_f32"])
        B.ishmem_int32_sum_reduce(B.ISHMEM_TEAM_WORLD, dst, src, S["reduce_i32"])
        # the four halo signal words of every PE back to zero: one put-to-self from the zeroed end of src
        B.ishmemx_putmem_spmd(jsig, zeros, 32, 0, B.ISHMEMX_WORK_GROUP, 32, 1)
        B.ishmemx_jacobi(jb0, jb1, jsig, S["jacobi_n"], S["jacobi_n"], S["jacobi_sweeps"], 1,
                         args.jacobi_groups, 0, res)
        B.ishmem_barrier_all()

    for _ in range(max(args.warmup, 3)):
        step(False)
    status = B.ishmemx_status(1)
    if status:
        raise SystemExit(f"device status {status} after warm-up")

    visible = [v for v in os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",") if v.strip()]
    sampler = ClockSampler(visible[local_rank] if local_rank < len(visible) else local_rank)
    replicas.barrier()
    torch.cuda.synchronize()
    sampler.start()
    launches0 = B.ishmemx_launch_count()
    t_start, t_end = ev(), ev()
    t_start.record(team_stream)
    for _ in range(args.steps):
        step(True)
    t_end.record(team_stream)
    torch.cuda.synchronize()
    replicas.barrier()
    clocks = sampler.stop()
    launches = B.ishmemx_launch_count() - launches0
    local_ms = t_start.elapsed_time(t_end)
    total_step_bytes = sum(nbytes.values())
    rate, ms = replicas.whole_job_rate(total_step_bytes * args.steps, local_ms)
    status = B.ishmemx_status(1)

    put_ms = float(np.mean([a.elapsed_time(b) for a, b in put_ev]))
    get_ms = float(np.mean([a.elapsed_time(b) for a, b in get_ev]))
    peaks = measured_peaks()
    achieved = nbytes["put"] / (put_ms * 1e-3) / 1e9
    roof = {"bound": "hbm", "kernel": f"k_rma<{args.level}> work-group put ({KERNEL_FORM[args.level]}), ring pattern, "
                                      f"{S['put'] // MiB} MiB/PE x {NPES} PEs",
            "achieved": round(achieved, 1), "peak": peaks["hbm_gbs"], "peak_source": peaks["source"],
            "unit": "GB/s", "frac": round(achieved / peaks["hbm_gbs"], 4),
            "frac_of_nominal_8TBs": round(achieved / 8000.0, 4), "traffic": TRAFFIC_PER_LAUNCH.get(args.level),
            "ms_per_launch": round(put_ms, 4),
            "get_achieved": round(nbytes["get"] / (get_ms * 1e-3) / 1e9, 1)}

    out = {"metric": "put/get & reduce GB/s (algorithmic bytes of one whole hot-path step / device time)",
           "value": round(rate / 1e9, 2), "unit": "GB/s", "n_gpus": world, "steps": args.steps,
           "warmup": max(args.warmup, 3), "ms_per_step": round(ms / args.steps, 4),
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8",
           "data": "synthetic", "gpu_launches": int(launches), "device_status": int(status),
           "config": {"workload": "configs[1]: 8 logical PEs x 512 MiB symmetric heap, ring pattern, "
                                  "256 MiB put/get messages per PE plus one pass of every other hot-path op",
                      "npes": NPES, "heap_bytes_per_pe": HEAP, "step_bytes": nbytes,
                      "level": args.level, "threads": args.threads, "groups_per_pe": args.groups,
                      "l2": "inputs (4 GiB) larger than L2; no flush", "parallelism": f"replicas x{world}"},
           "roofline": roof, "clocks": clocks,
           "pingpong_half_rtt_us": round(float(rtt[0]) / 1e3, 3)}

    if not args.no_breakdown and rank == 0:
        out["breakdown"] = breakdown(B, torch, team_stream, locals())
    if not args.no_e2e:
        out["e2e"] = e2e(B, torch, replicas, dst, src, level, args, world)
    if rank == 0 and world == 1 and not args.no_cpu:
        out["cpu_baseline"] = cpu_baseline(args.cpu_scale, reps=5)
    B.ishmem_finalize()
    del heap
    torch.cuda.empty_cache()
    if rank == 0 and not args.no_breakdown:
        # the other two bandwidth configurations, outside the timed step (12 PEs each, own sessions)
        out["config5_jacobi"] = config5_leg(B, torch, peaks)
        out["config3_collectives"] = config3_leg(B, torch, peaks)
    replicas.finalize()
    return out if rank == 0 else {}


def config5_leg(B, torch, peaks) -> dict:
    """configs[4]: 12 PEs, 16384 x 16384 float64 Jacobi with in-kernel put_signal halos, in the launch
    shape the library picks (six sweeps per launch).  48 sweeps timed after an untimed call.  The
    fraction is taken at the bytes a launch has to move: 16 B per cell per LAUNCH."""
    npes, n, sweeps = 12, 16384, 48
    rows_max = -(-n // npes)
    nbytes = (rows_max + 2) * n * 8
    heap_bytes = 2 * nbytes + 2 * MiB     # the buffers, the signals and the call's own halo rows
    heap = torch.zeros(npes * heap_bytes, dtype=torch.uint8, device="cuda")
    B.ishmemx_init_external(npes, heap_bytes, heap.data_ptr())
    ts = torch.cuda.Stream()
    B.ishmemx_set_stream(-1, ts.cuda_stream)
    b0, b1, sig = B.ishmem_malloc(nbytes), B.ishmem_malloc(nbytes), B.ishmem_calloc(4, 8)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(4)
    base, extra = divmod(n, npes)
    for p in range(npes):                              # uniform [0, 1) interior, zero ring (config 5's recipe)
        rows = base + (1 if p < extra else 0)
        strip = heap[p * heap_bytes + (b0 - heap.data_ptr()):][:nbytes].view(torch.float64).view(rows_max + 2, n)
        strip[1:rows + 1].uniform_(0.0, 1.0, generator=gen)
        strip[:, 0] = 0
        strip[:, n - 1] = 0
        if p == 0:
            strip[1] = 0
        if p == npes - 1:
            strip[rows] = 0
    torch.cuda.synchronize()
    res = np.zeros(1)
    out = {}
    for name, fuse, per_launch in (("six_sweeps_per_launch", 1, 6), ("four_sweeps_per_launch", 4, 4), ("one_sweep_per_launch", 0, 1)):
        B.ishmemx_set_option(B.ISHMEMX_OPT_JACOBI_FUSE, fuse)
        best = 1e30
        for rep in range(3):
            for p in range(npes):
                for w in range(4):
                    B.ishmem_uint64_p(p, sig + 8 * w, 0, p)
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(ts)
            B.ishmemx_jacobi(b0, b1, sig, n, n, sweeps, 1, 12, 0, res)
            b.record(ts)
            torch.cuda.synchronize()
            if rep:                                    # the first call loads the kernels
                best = min(best, a.elapsed_time(b))
        us = best * 1e3 / sweeps
        moved = 16.0 * n * n / per_launch / (us * 1e-6) / 1e9
        out[name] = {"us_per_sweep": round(us, 2), "us_per_launch": round(us * per_launch, 1),
                     "GB/s_at_16B_per_cell_per_sweep": round(16.0 * n * n / (us * 1e-6) / 1e9, 1),
                     "GB/s_moved": round(moved, 1), "frac_of_copy_peak_at_bytes_moved": round(moved / peaks["hbm_gbs"], 4)}
    out["workload"] = f"{npes} PEs, {n} x {n} float64, {sweeps} sweeps per call, best of 2 timed calls"
    out["device_status"] = int(B.ishmemx_status(1))
    B.ishmem_finalize()
    del heap
    torch.cuda.empty_cache()
    return out


def config3_leg(B, torch, peaks) -> dict:
    """configs[2] at large counts: 12 PEs, float32 sum_reduce of 64 Mi elements, broadcast of 256 MiB from
    root 0, fcollect of 16 Mi float32 per PE; algorithmic bytes (2 P n s; n + P n; P n + P^2 n) over the
    best of 5 launches."""
    npes, n_red, n_bc, n_fc = 12, 64 << 20, 256 * MiB, 64 * MiB
    heap_bytes = n_bc + npes * n_fc + MiB
    heap = torch.empty(npes * heap_bytes, dtype=torch.uint8, device="cuda")
    heap.view(torch.float32).normal_(generator=torch.Generator(device="cuda").manual_seed(2))
    B.ishmemx_init_external(npes, heap_bytes, heap.data_ptr())
    ts = torch.cuda.Stream()
    B.ishmemx_set_stream(-1, ts.cuda_stream)
    src, dst = B.ishmem_malloc(n_bc), B.ishmem_malloc(npes * n_fc)
    W = B.ISHMEM_TEAM_WORLD
    ops = {"sum_reduce_f32": (lambda: B.ishmem_float_sum_reduce(W, dst, src, n_red), 2 * npes * 4 * n_red),
           "broadcast": (lambda: B.ishmem_broadcastmem(W, dst, src, n_bc, 0), n_bc * (1 + npes)),
           "fcollect": (lambda: B.ishmem_fcollectmem(W, dst, src, n_fc), n_fc * (npes + npes * npes))}
    out = {}
    for name, (fn, nbytes) in ops.items():
        best = 1e30
        for rep in range(6):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record(ts)
            fn()
            b.record(ts)
            torch.cuda.synchronize()
            if rep:
                best = min(best, a.elapsed_time(b))
        g = nbytes / (best * 1e-3) / 1e9
        out[name] = {"ms": round(best, 4), "GB/s": round(g, 1), "frac_of_copy_peak": round(g / peaks["hbm_gbs"], 4)}
    out["workload"] = (f"{npes} PEs; sum_reduce {n_red} float32, broadcast {n_bc // MiB} MiB, "
                       f"fcollect {n_fc // MiB} MiB per PE")
    out["device_status"] = int(B.ishmemx_status(1))
    B.ishmem_finalize()
    del heap
    torch.cuda.empty_cache()
    return out


# DRAM bytes per launch of the put kernel: ncu capture of the 8 x 32 MiB case (reads scale with the
# bytes copied; writes are the algorithmic bytes minus the ~52 MB tail that stays in L2)
TRAFFIC_PER_LAUNCH = {"tiled": 4.24e9, "bulk": 4.24e9, "ldst": None}
KERNEL_FORM = {"tiled": "loads/stores, one 32 KiB tile per block", "bulk": "TMA ring, resident blocks",
               "ldst": "loads/stores, resident blocks"}


def breakdown(B, torch, team_stream, env) -> dict:
    """Per-op device time of one step's ops, each timed alone (5 repeats, best), GB/s of its
    algorithmic bytes, and Mops/s for the atomics."""
    S, nbytes = env["S"], env["nbytes"]
    src, dst, level, args = env["src"], env["dst"], env["level"], env["args"]
    word, inc, fetched = env["word"], env["inc"], env["fetched"]
    cword, ccond, cval, table = env["cword"], env["ccond"], env["cval"], env["table"]

    def timed(fn, reps=5):
        best = 1e30
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record(team_stream)
            fn()
            b.record(team_stream)
            torch.cuda.synchronize()
            best = min(best, a.elapsed_time(b))
        return best

    W = B.ISHMEM_TEAM_WORLD
    ops = {
        "put": lambda: B.ishmemx_putmem_spmd(dst, src, S["put"], 1, level, args.threads, args.groups),
        "get": lambda: B.ishmemx_getmem_spmd(dst, src, S["get"], 1, level, args.threads, args.groups),
        "copy_engine_put": lambda: B.ishmemx_putmem_spmd_copy_engine(dst, src, S["put"], 1),
        "broadcast": lambda: B.ishmem_broadcastmem(W, dst, src, S["bcast"], 0),
        "fcollect": lambda: B.ishmem_fcollectmem(W, dst, src, S["fcollect"]),
        "reduce_f32": lambda: B.ishmem_float_sum_reduce(W, dst, src, S["reduce_f32"]),
        "fetch_add": lambda: B.ishmemx_int64_atomic_fetch_add_batch(table, word, inc, fetched, NOPS_FADD, 1024, 2),
        "fetch_add_warp_aggregation": lambda: B.ishmemx_int64_atomic_fetch_add_batch(table, word, inc, fetched,
                                                                                       NOPS_FADD, 256, 1),
        "fetch_add_no_aggregation": lambda: B.ishmemx_int64_atomic_fetch_add_batch(table, word, inc, fetched,
                                                                                     NOPS_FADD, 256, 0),
        "compare_swap": lambda: B.ishmemx_int64_atomic_compare_swap_batch(table, cword, ccond, cval, fetched,
                                                                          NOPS_CAS, 256, 1),
        "compare_swap_no_aggregation": lambda: B.ishmemx_int64_atomic_compare_swap_batch(table, cword, ccond, cval,
                                                                                         fetched, NOPS_CAS, 256, 0),
        "jacobi": lambda: (B.ishmemx_putmem_spmd(env["jsig"], env["zeros"], 32, 0, B.ISHMEMX_WORK_GROUP, 32, 1),
                           B.ishmemx_jacobi(env["jb0"], env["jb1"], env["jsig"], S["jacobi_n"], S["jacobi_n"],
                                            S["jacobi_sweeps"], 1, args.jacobi_groups, 0, None)),
    }
    res = {}
    for name, fn in ops.items():
        ms = timed(fn)
        key = {"copy_engine_put": "put", "fetch_add_no_aggregation": "fetch_add",
               "fetch_add_warp_aggregation": "fetch_add", "compare_swap_no_aggregation": "compare_swap"}.get(name, name)
        entry = {"ms": round(ms, 4), "GB/s": round(nbytes[key] / (ms * 1e-3) / 1e9, 1)}
        if "fetch_add" in name:
            entry["Mops/s"] = round(NOPS_FADD / (ms * 1e-3) / 1e6, 1)
        if name.startswith("compare_swap"):
            entry["Mops/s"] = round(NOPS_CAS / (ms * 1e-3) / 1e6, 1)
        res[name] = entry
    return res


def e2e(B, torch, replicas, dst, src, level, args, world) -> dict:
    """Same ring put through the C ABI with HOST buffers: every step copies the 8 payloads
    from pinned host memory into the PEs' sources, runs the put, and reads the 8
    destinations back (ishmemx_host_put_ring)."""
    n = args.e2e_bytes
    hsrc = torch.empty(NPES * n, dtype=torch.uint8).pin_memory()
    hdst = torch.empty(NPES * n, dtype=torch.uint8).pin_memory()
    hsrc.view(torch.int64).copy_(torch.arange(NPES * n // 8, dtype=torch.int64))
    for _ in range(2):
        B.ishmemx_host_put_ring(hdst.data_ptr(), hsrc.data_ptr(), dst, src, n, 1, level, args.threads, args.groups)
    steps = max(2, min(args.steps, 5))
    replicas.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        B.ishmemx_host_put_ring(hdst.data_ptr(), hsrc.data_ptr(), dst, src, n, 1, level, args.threads, args.groups)
    torch.cuda.synchronize()
    local_ms = (time.perf_counter() - t0) * 1e3
    ok = bool(torch.equal(hdst[n:2 * n], hsrc[0:n]))          # PE 1 received PE 0's payload
    rate, ms = replicas.whole_job_rate(2 * n * NPES * steps, local_ms)
    # what the bus alone gives for the same bytes: plain pinned copies of NPES * n bytes each way, both
    # directions at once on two streams (the end-to-end call overlaps them between PEs), and each alone
    dev_in = torch.empty(NPES * n, dtype=torch.uint8, device="cuda")
    dev_out = torch.empty(NPES * n, dtype=torch.uint8, device="cuda")
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()

    def copies(h2d, d2h):
        best = 1e30
        for _ in range(3):
            torch.cuda.synchronize()
            t = time.perf_counter()
            if h2d:
                with torch.cuda.stream(s_in):
                    dev_in.copy_(hsrc, non_blocking=True)
            if d2h:
                with torch.cuda.stream(s_out):
                    hdst.copy_(dev_out, non_blocking=True)
            torch.cuda.synchronize()
            best = min(best, time.perf_counter() - t)
        return best

    t_both, t_in, t_out = copies(True, True), copies(True, False), copies(False, True)
    bus = 2 * n * NPES / t_both / 1e9
    return {"value": round(rate / 1e9, 2), "unit": "GB/s", "h2d_bytes_per_step": NPES * n,
            "d2h_bytes_per_step": NPES * n, "ms_per_step": round(ms / steps, 3), "steps": steps,
            "call": "ishmemx_host_put_ring (pinned host buffers -> heap -> work-group put ring -> host)",
            "verified": ok,
            "pcie_copy_only": {"both_directions_GB/s": round(bus, 2), "h2d_alone_GB/s": round(n * NPES / t_in / 1e9, 2),
                               "d2h_alone_GB/s": round(n * NPES / t_out / 1e9, 2),
                               "note": "plain pinned cudaMemcpyAsync of the same bytes, no put, this rank"},
            "frac_of_pcie_copy_only": round(local_rate_gbs(2 * n * NPES * steps, local_ms) / bus, 3)}


def local_rate_gbs(nbytes, ms):
    return nbytes / (ms * 1e-3) / 1e9


def measured_peaks() -> dict:
    f = ROOT / "MEASURED_PEAKS.json"
    if f.exists():
        d = json.loads(f.read_text())
        return {"hbm_gbs": float(d["hbm_gbs"]), "source": "measured (MEASURED_PEAKS.json)"}
    return {"hbm_gbs": 6650.0, "source": "fallback (earlier measurement on this pool)"}


# ------------------------------------------------------------------------ CPU arm ---

def oracle_step(O, scale: int, state: dict) -> float:
    """One pass of the same op list on the CPU oracle at 1/scale sizes; returns seconds."""
    import oracle as orc
    from paper_2409_20476_b200 import inputs

    S = sizes(scale)
    o = state.get("o")
    if o is None:
        heap = 2 * S["put"] + (1 << 16)
        o = O(NPES, heap)
        state["o"] = o
        state["src"] = o.malloc(S["put"])
        state["dst"] = o.malloc(S["put"])
        for p in range(NPES):
            o.view(state["src"], S["put"], p)[:] = np.resize(inputs.byte_payload(inputs.SEED_C2, p, MiB), S["put"])
        state["word"] = inputs.zipf_indices(inputs.SEED_C4, 0, S["fadd_ops"], NWORDS_FADD)
        state["inc"] = inputs.increments(inputs.SEED_C4, 0, S["fadd_ops"])
        state["cword"] = inputs.zipf_indices(inputs.SEED_C4, 1, S["cas_ops"], NWORDS_CAS)
        state["ccond"] = np.zeros(S["cas_ops"], dtype=np.int64)
        state["cval"] = np.arange(1, S["cas_ops"] + 1, dtype=np.int64)
        state["grid"] = inputs.jacobi_grid(inputs.SEED_C5, S["jacobi_n"], S["jacobi_n"])
    src, dst = state["src"], state["dst"]
    t0 = time.perf_counter()
    for p in range(NPES):
        o.putmem(p, dst, o.ptr(src, S["put"], p), S["put"], (p + 1) % NPES)
    for p in range(NPES):
        o.getmem(p, o.ptr(dst, S["get"], p), src, S["get"], (p + 1) % NPES)
    for p in range(NPES):
        o.putmem(p, dst, o.ptr(src, S["work_item"], p), S["work_item"], (p + 1) % NPES)
        o.putmem(p, dst, o.ptr(src, S["sub_group"], p), min(S["sub_group"], S["put"]), (p + 2) % NPES)
    o.p(dst, np.int64(1), 1)
    for p in range(NPES):
        o.putmem(p, dst, o.ptr(src, S["nbi"], p), S["nbi"], (p + 1) % NPES)
    o.putmem_signal(0, dst + 4096, o.ptr(src, S["signal"], 0), S["signal"], dst, 1, orc.SIG_SET, 1)
    o.test(1, dst, orc.C_GE, 1)
    for r in range(S["pp_rounds"]):
        o.putmem_signal(0, dst + 8192, o.ptr(dst + 8192, S["pp_bytes"], 0), S["pp_bytes"], dst + 64, r + 1, orc.SIG_SET, 1)
        o.putmem_signal(1, dst + 8192, o.ptr(dst + 8192, S["pp_bytes"], 1), S["pp_bytes"], dst + 64, r + 1, orc.SIG_SET, 0)
    o.fetch_add_batch(dst, state["word"], state["inc"])
    o.compare_swap_batch(dst, state["cword"], state["ccond"], state["cval"])
    o.broadcastmem(o.world, dst, src, S["bcast"], 0)
    o.fcollectmem(o.world, dst, src, S["fcollect"])
    o.reduce(o.world, dst, src, S["reduce_f32"], orc.R_SUM, orc.T_FLOAT)
    o.reduce(o.world, dst, src, min(S["reduce_i32"], S["put"] // 4), orc.R_SUM, orc.T_INT32)
    orc.jacobi(state["grid"], S["jacobi_sweeps"])
    return time.perf_counter() - t0


def sample_bytes(scale: int) -> int:
    S = sizes(scale)
    b = step_bytes(S)
    b["sub_group"] = 2 * min(S["sub_group"], S["put"]) * NPES
    b["reduce_i32"] = 2 * NPES * 4 * min(S["reduce_i32"], S["put"] // 4)
    return sum(b.values())


def cpu_model() -> str:
    try:
        for line in open("/proc/cpuinfo"):
            if line.lower().startswith("model name"):
                return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def oracle_threaded(O, scale: int, state: dict, pool, nthreads: int) -> tuple[float, int]:
    """The bandwidth ops of the step on the unchanged oracle, called from `nthreads` host threads where
    the op is trivially parallel (ctypes releases the interpreter lock inside the C calls): per-PE puts and
    gets concurrently, reduce / broadcast / fcollect cut into element ranges, Jacobi sweeps cut into bands
    of rows (each band one single-sweep call on its rows plus one row above and below, which the call
    keeps fixed).  Results are those of the sequential calls by construction.  Returns (seconds, bytes)."""
    import oracle as orc
    S = sizes(scale)
    o, src, dst = state["o"], state["src"], state["dst"]
    b = step_bytes(S)
    P = NPES

    def ranges(n, unit):
        per = -(-n // nthreads)
        per = -(-per // unit) * unit
        return [(lo, min(n, lo + per)) for lo in range(0, n, per)]

    t0 = time.perf_counter()
    list(pool.map(lambda p: o.putmem(p, dst, o.ptr(src, S["put"], p), S["put"], (p + 1) % P), range(P)))
    list(pool.map(lambda p: o.getmem(p, o.ptr(dst, S["get"], p), src, S["get"], (p + 1) % P), range(P)))
    list(pool.map(lambda p: o.putmem(p, dst, o.ptr(src, S["nbi"], p), S["nbi"], (p + 1) % P), range(P)))
    list(pool.map(lambda r: o.broadcastmem(o.world, dst + r[0], src + r[0], r[1] - r[0], 0), ranges(S["bcast"], 64)))
    # fcollect in element ranges would change the layout of dest: one call per source PE's block instead
    list(pool.map(lambda i: [o.putmem(i, dst + i * S["fcollect"], o.ptr(src, S["fcollect"], i), S["fcollect"], q)
                             for q in range(P)], range(P)))
    list(pool.map(lambda r: o.reduce(o.world, dst + 4 * r[0], src + 4 * r[0], r[1] - r[0], orc.R_SUM, orc.T_FLOAT),
                  ranges(S["reduce_f32"], 16)))
    g = state["grid"]
    ny = g.shape[0]
    a = g.copy()
    for _ in range(S["jacobi_sweeps"]):
        nxt = a.copy()

        def band(r, a=a, nxt=nxt):
            lo, hi = max(r[0], 1), min(r[1], ny - 1)
            if lo < hi:
                nxt[lo:hi] = orc.jacobi(a[lo - 1:hi + 1], 1)[0][1:-1]
        list(pool.map(band, ranges(ny, 1)))
        a = nxt
    dt = time.perf_counter() - t0
    nbytes = b["put"] + b["get"] + b["nbi"] + b["broadcast"] + b["fcollect"] + b["reduce_f32"] + b["jacobi"]
    return dt, nbytes


def cpu_baseline(scale: int, reps: int) -> dict:
    from concurrent.futures import ThreadPoolExecutor
    from oracle import Oracle
    state: dict = {}
    best = min(oracle_step(Oracle, scale, state) for _ in range(reps))
    nproc = os.cpu_count() or 1
    nthreads = min(nproc, 64)
    with ThreadPoolExecutor(max_workers=nthreads) as pool:
        runs = [oracle_threaded(Oracle, scale, state, pool, nthreads) for _ in range(3)]
    t_thr, b_thr = min(runs)
    return {"value": round(sample_bytes(scale) / best / 1e9, 3), "unit": "GB/s", "cores": 1,
            "kind": "oracle", "seconds": round(best, 2),
            "sample": f"one step of the same op list at 1/{scale} of the sizes "
                      f"({sample_bytes(scale) / 2**30:.2f} GiB algorithmic), sequential CPU oracle, best of {reps}",
            "nproc": nproc, "cpu_model": cpu_model(),
            "threaded": {"value": round(b_thr / t_thr / 1e9, 3), "unit": "GB/s", "cores": nthreads,
                         "seconds": round(t_thr, 2),
                         "sample": f"the bandwidth ops of the same step (put, get, nbi put, broadcast, fcollect, float32 "
                                   f"sum_reduce, Jacobi: {b_thr / 2**30:.2f} GiB algorithmic) on the unchanged oracle "
                                   f"called from {nthreads} host threads, best of 3"}}


def run_reference(args) -> dict:
    from paper_2409_20476_b200 import replicas
    rank, _, world = replicas.env_world()
    if rank != 0:
        return {}
    from oracle import Oracle
    state: dict = {}
    scale = args.cpu_scale
    for _ in range(min(args.warmup, 1)):
        oracle_step(Oracle, scale, state)
    steps = max(1, min(args.steps, 3))
    t = [oracle_step(Oracle, scale, state) for _ in range(steps)]
    total = sum(t)
    val = round(sample_bytes(scale) * steps / total / 1e9, 3)
    sample = (f"each step = the same op list at 1/{scale} of the sizes "
              f"({sample_bytes(scale) / 2**30:.2f} GiB algorithmic)")
    return {"impl": "reference",
            "metric": "put/get & reduce GB/s (algorithmic bytes of one whole hot-path step / device time)",
            "value": val, "unit": "GB/s", "n_gpus": world, "steps": steps, "warmup": min(args.warmup, 1),
            "ms_per_step": round(total / steps * 1e3, 2), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "u8", "data": "synthetic",
            "config": {"workload": "configs[1] (8 logical PEs, ring pattern), bounded CPU sample", "sample": sample},
            "cpu_baseline": {"value": val, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def run_plumbing(args) -> dict:
    """The multi-rank plumbing alone (no GPU work): rendezvous, barrier, sum and max over ranks on made-up
    figures -- rank r 'processed' (r + 1) * 100 units in (r + 1) * 10 ms.  Runs on CPU over gloo."""
    from paper_2409_20476_b200 import replicas
    rank, _, world = replicas.init(backend="gloo")
    replicas.barrier()
    rate, ms = replicas.whole_job_rate((rank + 1) * 100.0, (rank + 1) * 10.0)
    replicas.barrier()
    replicas.finalize()
    return {"impl": "plumbing", "n_gpus": world, "value": rate, "ms_per_step": ms} if rank == 0 else {}


def run_profile_case(args) -> dict:
    """A small case of one kernel for profiler captures: 8 PEs, `--msg-mib` per PE (default
    32 MiB: 512 MiB of sources + destinations, larger than L2, far below a GiB), a few
    launches of the named op and nothing else."""
    import torch
    from paper_2409_20476_b200 import binding as B
    from paper_2409_20476_b200 import inputs

    if args.profile_case in ("jacobi", "jacobi_persistent"):
        return run_profile_jacobi(args)
    n = args.msg_mib * MiB
    heap_bytes = 2 * n + (1 << 20) if args.profile_case != "fcollect" else (NPES + 1) * n + (1 << 20)
    heap = torch.empty(NPES * heap_bytes, dtype=torch.uint8, device="cuda")
    blk = torch.from_numpy(inputs.normal_values(inputs.SEED_C3, 0, MiB // 4, np.float32)).cuda().view(torch.uint8)
    heap.view(-1, MiB)[:] = blk
    B.ishmemx_init_external(NPES, heap_bytes, heap.data_ptr())
    src = B.ishmem_malloc(n)
    dst = B.ishmem_malloc(n if args.profile_case != "fcollect" else NPES * n)
    level = {"tiled": B.ISHMEMX_WORK_GROUP, "bulk": B.ISHMEMX_WORK_GROUP_BULK, "ldst": B.ISHMEMX_WORK_GROUP}[args.level]
    W = B.ISHMEM_TEAM_WORLD
    op = {
        "put": lambda: B.ishmemx_putmem_spmd(dst, src, n, 1, level, args.threads, args.groups),
        "get": lambda: B.ishmemx_getmem_spmd(dst, src, n, 1, level, args.threads, args.groups),
        "reduce": lambda: B.ishmem_float_sum_reduce(W, dst, src, n // 4),
        "broadcast": lambda: B.ishmem_broadcastmem(W, dst, src, n, 0),
        "fcollect": lambda: B.ishmem_fcollectmem(W, dst, src, n),
    }[args.profile_case]
    ts = torch.cuda.Stream()
    B.ishmemx_set_stream(-1, ts.cuda_stream)
    times = []
    for _ in range(3 + args.steps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(ts)
        op()
        b.record(ts)
        torch.cuda.synchronize()
        times.append(a.elapsed_time(b))
    B.ishmem_finalize()
    return {"profile_case": args.profile_case, "msg_mib": args.msg_mib, "ms": [round(t, 4) for t in times[3:]]}


def run_profile_jacobi(args) -> dict:
    """Small Jacobi case for profiler captures: 8 PEs, 4096 x 16384 float64 (full-width rows as in config 5,
    two buffers of 512 MiB: larger than L2, and enough blocks for the launch shape used at full size),
    `--steps` calls of 12 sweeps each (two launches of six sweeps)."""
    import torch
    from paper_2409_20476_b200 import binding as B
    from paper_2409_20476_b200 import inputs

    ny, nx, sweeps = 4096, 16384, 12
    persistent = args.profile_case == "jacobi_persistent"   # the resident kernel, strips cut by column tiles
    rows = ny // NPES
    nbytes = (rows + 2) * nx * 8
    heap_bytes = 2 * nbytes + 2 * MiB     # the buffers, the signals and the call's own halo rows
    heap = torch.zeros(NPES * heap_bytes, dtype=torch.uint8, device="cuda")
    B.ishmemx_init_external(NPES, heap_bytes, heap.data_ptr())
    b0, b1, sig = B.ishmem_malloc(nbytes), B.ishmem_malloc(nbytes), B.ishmem_calloc(4, 8)
    grid = inputs.jacobi_grid(inputs.SEED_C5, ny, nx)
    for p in range(NPES):
        o = p * heap_bytes + (b0 - heap.data_ptr()) + nx * 8
        heap[o:o + rows * nx * 8].copy_(torch.from_numpy(grid[p * rows:(p + 1) * rows].view(np.uint8).ravel()))
    torch.cuda.synchronize()
    ts = torch.cuda.Stream()
    B.ishmemx_set_stream(-1, ts.cuda_stream)
    res, times = np.zeros(1), []
    if persistent:
        B.ishmemx_set_option(B.ISHMEMX_OPT_JACOBI_SPLIT, 2)
    for _ in range(2 + args.steps):
        for p in range(NPES):
            for w in range(4):
                B.ishmem_uint64_p(p, sig + 8 * w, 0, p)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(ts)
        B.ishmemx_jacobi(b0, b1, sig, ny, nx, sweeps, 1, args.jacobi_groups, 0, res)
        b.record(ts)
        torch.cuda.synchronize()
        times.append(a.elapsed_time(b))
    status = B.ishmemx_status(1)
    B.ishmem_finalize()
    return {"profile_case": args.profile_case, "ny": ny, "nx": nx, "sweeps_per_call": sweeps, "status": status,
            "ms": [round(t, 4) for t in times[2:]]}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--profile-case", default=None, choices=["put", "get", "reduce", "broadcast", "fcollect", "jacobi", "jacobi_persistent"],
                    help="run only a few launches of one kernel on a small case (for ncu captures)")
    ap.add_argument("--msg-mib", type=int, default=32)
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference", "plumbing"],
                    help="ours: the CUDA library; reference: the CPU oracle on a bounded sample; plumbing: the "
                         "multi-rank rendezvous / barrier / max-over-ranks path alone, on CPU")
    ap.add_argument("--level", default="tiled", choices=["tiled", "bulk", "ldst"],
                    help="tiled: loads/stores, one tile per block (the library's own choice for large messages); "
                         "bulk / ldst: resident blocks (--groups per PE) with the TMA ring / loads and stores")
    ap.add_argument("--threads", type=int, default=256)
    ap.add_argument("--groups", type=int, default=37, help="work-groups per PE in the put/get launch")
    ap.add_argument("--jacobi-groups", type=int, default=18)
    ap.add_argument("--cpu-scale", type=int, default=1)
    ap.add_argument("--e2e-bytes", type=int, default=64 * MiB, help="payload per PE of the end-to-end leg")
    ap.add_argument("--no-breakdown", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    if args.level == "tiled":
        args.groups = 0  # the library sizes the grid: one tile of threads x 128 bytes per block
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.profile_case:
        # started by hand (python bench.py --gpus N) rather than by torchrun: this process starts the N
        # ranks itself, one replica per device, and passes on what rank 0 prints
        from paper_2409_20476_b200 import replicas
        text, rc = replicas.spawn(args.gpus, [sys.executable, str(Path(__file__).resolve())] + sys.argv[1:])
        sys.stdout.write(text)
        sys.exit(rc)
    if args.profile_case:
        out = run_profile_case(args)
    elif args.impl == "plumbing":
        out = run_plumbing(args)
    else:
        out = run_reference(args) if args.impl == "reference" else run_ours(args)
    if out:
        print(json.dumps(out))


if __name__ == "__main__":
    main()
