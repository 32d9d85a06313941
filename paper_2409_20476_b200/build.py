"""Builds ``libishmem.so`` (sm_100a) in-tree from ``csrc/*.cu`` with nvcc."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
LIB = PKG / "libishmem.so"
BUILD = PKG / "_build"

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I", str(ROOT / "include"), "-I", str(CSRC)]


def nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not Path(exe).exists():
        raise RuntimeError("nvcc not found: libishmem.so cannot be built")
    return exe


def sources() -> list[Path]:
    return sorted(CSRC.glob("*.cu"))


def deps_mtime() -> float:
    files = list(CSRC.glob("*")) + list((ROOT / "include").glob("*"))
    return max(f.stat().st_mtime for f in files)


def build(force: bool = False, verbose: bool = False, ptxas_info: bool = False) -> Path:
    if not force and LIB.exists() and LIB.stat().st_mtime >= deps_mtime():
        return LIB
    BUILD.mkdir(exist_ok=True)
    objs = []
    procs = []
    for src in sources():
        obj = BUILD / (src.stem + ".o")
        cmd = [nvcc(), *NVCC_FLAGS, "-c", str(src), "-o", str(obj)]
        if ptxas_info:
            cmd += ["-Xptxas", "-v"]
        if verbose:
            print(" ".join(cmd), file=sys.stderr)
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT)))
        objs.append(obj)
    failed = False
    for src, p in procs:
        out, _ = p.communicate()
        if out and (verbose or ptxas_info or p.returncode):
            sys.stderr.write(out.decode())
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    tmp = LIB.with_suffix(f".so.{os.getpid()}")
    subprocess.run([nvcc(), "-shared", "-o", str(tmp), *map(str, objs), "-lcudart_static", "-ldl",
                    "-lpthread", "-lrt"], check=True)
    os.replace(tmp, LIB)
    return LIB


def build_user_kernel_example(force: bool = False) -> Path:
    """Compiles tests/csrc/user_kernel.cu -- a kernel of a library USER, built only against the
    public headers -- into tests/libuser_kernel.so (used by the GPU tests)."""
    src = ROOT / "tests" / "csrc" / "user_kernel.cu"
    out = ROOT / "tests" / "libuser_kernel.so"
    newest = max(src.stat().st_mtime, max(f.stat().st_mtime for f in (ROOT / "include").glob("*")))
    if not force and out.exists() and out.stat().st_mtime >= newest:
        return out
    tmp = out.with_suffix(f".so.{os.getpid()}")
    subprocess.run([nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-shared",
                    "-Xcompiler", "-fPIC", "-I", str(ROOT / "include"), str(src), "-o", str(tmp), "-lcudart_static",
                    "-ldl", "-lpthread", "-lrt"], check=True)
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    build(force="--force" in sys.argv, verbose=True, ptxas_info="--ptxas" in sys.argv)
    build_user_kernel_example(force="--force" in sys.argv)
    print(LIB)
