"""Builds the native pieces in-tree (no JIT cache): the CUDA C-ABI library and the input
generator.

Each target is rebuilt only when one of its sources is newer than the shared object."""
from __future__ import annotations

import os
import shutil
import subprocess
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
INCLUDE = ROOT / "include"

LIB_CUDA = PKG / "libdsfacto.so"
LIB_CUDA_DEBUG = PKG / "libdsfacto_debug.so"
LIB_WORKLOADS = PKG / "_workloads_gen.so"

NVCC_ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]


def _stale(target: Path, sources) -> bool:
    if not target.exists():
        return True
    t = target.stat().st_mtime
    return any(Path(s).stat().st_mtime > t for s in sources)


def _run(cmd) -> None:
    proc = subprocess.run([str(c) for c in cmd], capture_output=True, text=True)
    if proc.returncode != 0:
        raise RuntimeError("build failed: %s\n%s\n%s" % (" ".join(map(str, cmd)), proc.stdout, proc.stderr))


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not Path(exe).exists():
        raise RuntimeError("nvcc not found; the CUDA library cannot be built")
    return exe


def build_cuda(force: bool = False, verbose_ptxas: bool = False, debug: bool = False) -> Path:
    """The C-ABI library.  debug=True builds libdsfacto_debug.so with -DDSFACTO_DEBUG: the stratum SGD kernel
    then checks every index it forms (rows, columns, chunk and run bounds); a failed check is recorded in
    the launch's error word and reported by dsfacto_epoch, nothing traps."""
    srcs = sorted(CSRC.glob("*.cu"))
    deps = srcs + sorted(CSRC.glob("*.cuh")) + sorted(CSRC.glob("*.h")) + sorted(INCLUDE.glob("*.h"))
    target = LIB_CUDA_DEBUG if debug else LIB_CUDA
    if force or _stale(target, deps):
        tmp = target.with_suffix(".so.tmp%d" % os.getpid())
        cmd = [_nvcc(), "-O3", "-std=c++17", "-lineinfo", *NVCC_ARCH, "-shared", "-Xcompiler",
               "-fPIC,-O3,-fopenmp,-Wall", "-I", INCLUDE, "-I", CSRC, "-o", tmp, *srcs, "-lgomp"]
        if debug:
            cmd[1:1] = ["-DDSFACTO_DEBUG"]
        if verbose_ptxas:
            cmd[1:1] = ["-Xptxas", "-v"]
        _run(cmd)
        os.replace(tmp, target)
    return target


def build_workloads(force: bool = False) -> Path:
    src = CSRC / "workloads_gen.c"
    if force or _stale(LIB_WORKLOADS, [src]):
        tmp = LIB_WORKLOADS.with_suffix(".so.tmp%d" % os.getpid())
        _run(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, src, "-lm"])
        os.replace(tmp, LIB_WORKLOADS)
    return LIB_WORKLOADS


def build_all(force: bool = False) -> None:
    build_workloads(force)
    build_cuda(force)
    build_cuda(force, debug=True)
