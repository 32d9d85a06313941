"""Multi-GPU plumbing for the benchmark: independent replicas, no data-path collective.

The library runs N logical PEs inside ONE GPU (nothing spans a second GPU), so with
several GPUs every rank runs the same workload on its own device.  ``torch.distributed``
is used only to line the ranks up (barrier) and to take the maximum of their device times.
"""
from __future__ import annotations

import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist


def env_world() -> tuple[int, int, int]:
    """(rank, local_rank, world_size) from the torchrun environment, or (0, 0, 1)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str | None = None) -> tuple[int, int, int]:
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        if backend is None:
            backend = "nccl" if torch.cuda.is_available() else "gloo"
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        kw = {}
        if backend == "nccl":
            kw["device_id"] = torch.device("cuda", local_rank)
        dist.init_process_group(backend=backend, rank=rank, world_size=world, **kw)
    return rank, local_rank, world


def barrier() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float) -> float:
    """Maximum of a per-rank scalar (device time in ms)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float) -> float:
    """Sum of a per-rank scalar (units of work processed)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_rate(local_units: float, local_ms: float) -> tuple[float, float]:
    """(units per second over all ranks, max time in ms): all ranks' units / slowest rank's time."""
    total = sum_over_ranks(local_units)
    ms = max_over_ranks(local_ms)
    return (total / (ms * 1e-3) if ms > 0 else 0.0), ms


def spawn(world: int, argv: list[str], extra_env: dict | None = None, timeout: float | None = None):
    """Starts `world` ranks of the command `argv` on this node, one per device (RANK, LOCAL_RANK,
    WORLD_SIZE and the rendezvous address set the way torchrun sets them), waits for all of them and
    returns (rank 0's standard output, the largest exit code).  The ranks' standard error goes to this
    process's; the other ranks' standard output is dropped (rank 0 alone reports)."""
    with socket.socket() as s:                      # a free port for the rendezvous
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        env.setdefault("NCCL_DEBUG", "INFO")        # the communicator's size and transport show in the log
        env.update(extra_env or {})
        procs.append(subprocess.Popen(argv, env=env, stdout=subprocess.PIPE if rank == 0 else subprocess.DEVNULL,
                                      stderr=sys.stderr, text=True))
    out, rc = "", 0
    for rank, p in enumerate(procs):
        o, _ = p.communicate(timeout=timeout)
        if rank == 0:
            out = o or ""
        rc = max(rc, abs(p.returncode))
    return out, rc


def finalize() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
