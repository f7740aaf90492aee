"""Compile the CUDA sources into the in-tree C-ABI library ``libw2a8.so``.

Usage: ``python -m paper_2508_06753_b200.build [--force] [--verbose]``.
nvcc cross-compiles for sm_100a, so this works on a machine without a GPU.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libw2a8.so")


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    # several processes (one per GPU) may get here at once: one builds, the others wait for it
    import fcntl
    with open(LIB + ".lock", "w") as lock:
        fcntl.flock(lock, fcntl.LOCK_EX)
        try:
            if not force and not _stale():
                return LIB
            tmp = LIB + f".tmp{os.getpid()}"
            common = [_nvcc(), "-std=c++17", "-O3", "-lineinfo",
                      "-gencode", "arch=compute_100a,code=sm_100a",
                      "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]
            if verbose:
                common[1:1] = ["-Xptxas", "-v"]
            common += os.environ.get("W2A8_NVCC_FLAGS", "").split()      # e.g. -D switches of the kernels
            # one object per source file, compiled side by side, then one link
            objdir = os.path.join(PKG, "build")
            os.makedirs(objdir, exist_ok=True)
            objs = [os.path.join(objdir, os.path.basename(src)[:-3] + f".{os.getpid()}.o") for src in sources()]
            procs = [subprocess.Popen(common + ["-c", src, "-o", obj]) for src, obj in zip(sources(), objs)]
            failed = [src for src, pr in zip(sources(), procs) if pr.wait() != 0]
            if failed:
                raise subprocess.CalledProcessError(1, "nvcc -c " + " ".join(failed))
            subprocess.run(common[:1] + ["-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-cudart", "static",
                                         "-o", tmp] + objs, check=True)
            for obj in objs:
                os.remove(obj)
            os.replace(tmp, LIB)        # atomic: nobody ever loads a half-written library
        finally:
            fcntl.flock(lock, fcntl.LOCK_UN)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
