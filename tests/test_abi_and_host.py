"""CPU-only checks of the boundary and the host logic: the C-ABI library loads and exports
every symbol the header declares, the binding covers them with matching arity, the product
and the oracle do not reach into one another, the byte accounting of the benchmark, and the
multi-rank (replicas) plumbing over gloo with world_size 2."""
import json
import os
import re
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))


def declared_functions():
    """(name, number of parameters) for every prototype in include/ishmem.h after preprocessing."""
    src = subprocess.run(["gcc", "-E", "-P", str(ROOT / "include" / "ishmem.h")], check=True,
                         capture_output=True, text=True).stdout
    out = {}
    for m in re.finditer(r"\b(ishmemx?_\w+)\s*\(([^()]*)\)\s*;", src):
        params = m.group(2).strip()
        out[m.group(1)] = 0 if params in ("", "void") else params.count(",") + 1
    return out


@pytest.fixture(scope="module")
def built():
    import __graft_entry__
    __graft_entry__.build()
    from paper_2409_20476_b200 import binding
    return binding


def test_library_exports_every_declared_symbol(built):
    decl = declared_functions()
    assert len(decl) > 150
    nm = subprocess.run(["nm", "-D", "--defined-only", str(built.LIB_PATH)], check=True,
                        capture_output=True, text=True).stdout
    exported = {ln.split()[-1] for ln in nm.splitlines() if " T " in ln}
    missing = sorted(set(decl) - exported)
    assert not missing, f"declared but not exported: {missing}"
    undeclared = sorted(n for n in exported if n.startswith("ishmem") and n not in decl)
    assert not undeclared, f"exported but not declared in include/ishmem.h: {undeclared}"


def test_binding_covers_header_with_matching_arity(built):
    decl = declared_functions()
    assert set(built.SIGNATURES) == set(decl)
    for name, (_, args) in built.SIGNATURES.items():
        assert len(args) == decl[name], name
    lib = built.lib()
    for name in decl:
        assert hasattr(lib, name)


def test_calls_before_init_fail_loudly(built):
    assert built.ishmem_n_pes() == 0
    with pytest.raises(built.IshmemError) as e:
        built.ishmem_putmem(0, 1, 1, 1, 0)
    assert e.value.code == built.ISHMEM_ERR_NOT_INITIALIZED
    with pytest.raises(built.IshmemError) as e:
        built.ishmem_barrier_all()
    assert e.value.code == built.ISHMEM_ERR_NOT_INITIALIZED
    assert built.ishmem_malloc(64) == 0 and built.ishmemx_ctx(0) == 0
    assert built.strerror(built.ISHMEM_ERR_TIMEOUT).startswith("a bounded")


def test_no_cpu_fallback_without_a_device(built):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(built.IshmemError) as e:
        built.ishmem_init(4, 1 << 20)
    assert e.value.code == built.ISHMEM_ERR_CUDA
    assert "no CPU path" in built.ishmemx_last_cuda_error().decode()


def test_product_and_oracle_do_not_touch_each_other():
    pkg = ROOT / "paper_2409_20476_b200"
    for f in list(pkg.glob("*.py")) + list((pkg / "csrc").glob("*")) + list((ROOT / "include").glob("*")):
        if f.is_file():
            text = f.read_text()
            assert not re.search(r"^\s*(import|from)\s+oracle\b", text, re.M), f
            assert "ishmem_oracle" not in text, f
    for f in (ROOT / "oracle").glob("*"):
        if f.suffix in (".py", ".c", ".h"):
            text = f.read_text()
            assert "paper_2409_20476_b200" not in text and "ishmem.h" not in text, f


def test_benchmark_byte_accounting():
    import bench
    S = bench.sizes()
    b = bench.step_bytes(S)
    MiB = 1 << 20
    assert b["put"] == 2 * 256 * MiB * 8 and b["get"] == b["put"]            # 2n per PE
    assert b["broadcast"] == 64 * MiB * 9                                    # n + P n
    assert b["fcollect"] == 16 * MiB * (8 + 64)                              # P n + P^2 n
    assert b["reduce_f32"] == 2 * 8 * 4 * 16 * MiB                           # 2 P n s
    assert b["jacobi"] == 16 * 4096 * 4096 * 4                               # 16 B per cell per sweep
    small = bench.sizes(16)
    assert small["put"] == 16 * MiB and small["jacobi_n"] % 8 == 0
    assert bench.sample_bytes(16) < sum(b.values()) // 8


def test_reference_arm_on_a_tiny_sample():
    """`bench.py --impl reference` times the CPU oracle and prints the contract's JSON line."""
    env = dict(os.environ, PYTHONPATH=str(ROOT))
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--cpu-scale", "64"], check=True, capture_output=True,
                         text=True, env=env, timeout=300).stdout
    line = json.loads(out.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["unit"] == "GB/s"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    # under a multi-rank launch only rank 0 works and prints
    env.update(RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2"],
                         check=True, capture_output=True, text=True, env=env, timeout=60).stdout
    assert out.strip() == ""


WORKER = r"""
import os, sys, json
sys.path.insert(0, sys.argv[1])
from paper_2409_20476_b200 import replicas
rank, local_rank, world = replicas.init(backend="gloo")
replicas.barrier()
# rank r processed (r+1)*100 units in (r+1)*10 ms
rate, ms = replicas.whole_job_rate((rank + 1) * 100.0, (rank + 1) * 10.0)
replicas.barrier()
print(json.dumps({"rank": rank, "world": world, "rate": rate, "ms": ms}))
replicas.finalize()
"""


def test_replicas_world_size_2_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = 29500 + os.getpid() % 2000
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script), str(ROOT)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    res = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err
        res.append(json.loads(out.strip().splitlines()[-1]))
    for r in res:
        assert r["world"] == 2
        assert r["ms"] == 20.0                       # max over ranks
        assert abs(r["rate"] - 300.0 / 0.020) < 1e-6  # all ranks' units / slowest rank's time


def test_bench_gpus_2_starts_two_ranks_by_itself():
    """`python bench.py --gpus 2` without a torchrun environment starts the two ranks itself: the
    plumbing arm (rendezvous over gloo, barrier, sum and max over ranks) reports a world of 2 and the
    whole-job figures, and the reference arm prints exactly one line, rank 0's, with n_gpus 2."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_PORT")}
    env["PYTHONPATH"] = str(ROOT)
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "plumbing", "--gpus", "2"], check=True,
                         capture_output=True, text=True, env=env, timeout=180).stdout
    lines = [ln for ln in out.strip().splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["ms_per_step"] == 20.0          # the slowest rank's time
    assert abs(line["value"] - 300.0 / 0.020) < 1e-6                     # all ranks' units over it
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                          "--warmup", "0", "--cpu-scale", "64"], check=True, capture_output=True, text=True, env=env,
                         timeout=300).stdout
    lines = [ln for ln in out.strip().splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0


def test_jacobi_launch_split_host_logic():
    """The launches of a Jacobi call: depths between 1 and the cap, deepest first, adding up to the sweep
    count, and as many as the sweep count is even or odd (each launch flips the buffers; the result must
    end where single sweeps leave it).  Long calls are all deepest launches but for a short tail."""
    import numpy as np
    from paper_2409_20476_b200 import binding as B
    for cap in (1, 2, 3, 4, 5, 6):
        for iters in list(range(0, 60)) + [199, 200, 201, 1000, 1001]:
            out = np.zeros(iters + 1, dtype=np.int32)
            n = B.ishmemx_jacobi_launch_depths(iters, cap, out, len(out))
            d = out[:n].tolist()
            assert sum(d) == iters and n % 2 == iters % 2, (cap, iters, d)
            assert all(1 <= k <= cap for k in d) and d == sorted(d, reverse=True), (cap, iters, d)
            if iters >= 40:
                assert d.count(cap) >= (iters - 24) // cap, (cap, iters, d)
    out = np.zeros(64, dtype=np.int32)
    assert B.ishmemx_jacobi_launch_depths(200, 4, out, 64) == 50 and set(out[:50].tolist()) == {4}
    assert B.ishmemx_jacobi_launch_depths(9, 4, out, 64) == 3 and out[:3].tolist() == [3, 3, 3]
    assert B.ishmemx_jacobi_launch_depths(8, 4, out, 64) == 2 and out[:2].tolist() == [4, 4]
    assert B.ishmemx_jacobi_launch_depths(5, 4, out, 64) == 3 and sum(out[:3].tolist()) == 5
    assert B.ishmemx_jacobi_launch_depths(5, 6, out, 64) == 1 and out[0] == 5
    assert B.ishmemx_jacobi_launch_depths(7, 4, None, 0) == 3          # count only
    assert B.ishmemx_jacobi_launch_depths(200, 6, out, 64) == 34 and out[:34].tolist().count(6) >= 30
    assert B.ishmemx_jacobi_launch_depths(12, 6, out, 64) == 2 and out[:2].tolist() == [6, 6]
    for bad in ((-1, 4), (5, 0), (5, 7)):
        assert B.ishmemx_jacobi_launch_depths(bad[0], bad[1], out, 64) == B.ISHMEM_ERR_ARG
