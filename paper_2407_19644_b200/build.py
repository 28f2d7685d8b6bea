"""Compile the CUDA library in-tree: paper_2407_19644_b200/libubp_b200.so (sm_100a).

    python -m paper_2407_19644_b200.build [--force] [--verbose] [--debug]

--debug builds libubp_b200_debug.so instead: the same library with -DUBP_DEBUG, in which the kernels compare every index
they take from the plan or compute for shared / global memory with its extent, report a failure through the plan's status
word and skip the access (nothing traps). Load it by setting UBP_B200_LIBRARY to its path before the package is imported.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libubp_b200.so")
LIB_DEBUG = os.path.join(HERE, "libubp_b200_debug.so")     # the checked build (-DUBP_DEBUG): same entry points
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")) + glob.glob(os.path.join(CSRC, "*.cpp")))


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.inc")) + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    lib = LIB_DEBUG if debug else LIB
    if not force and not _stale(lib):
        return lib
    objdir = os.path.join(HERE, "build_debug" if debug else "build")
    os.makedirs(objdir, exist_ok=True)
    common = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    common += os.environ.get("UBP_NVCC_FLAGS", "").split()      # extra flags, e.g. -DNAME for a diagnostic build
    if debug:
        common += ["-DUBP_DEBUG"]
    if verbose:
        common += ["-Xptxas", "-v"]
    objs = []
    procs = []
    for src in sources():
        obj = os.path.join(objdir, os.path.basename(src) + ".o")
        objs.append(obj)
        cmd = [NVCC, "-c", "-x", "cu" if src.endswith(".cu") else "c++", src, "-o", obj] + common
        procs.append((src, subprocess.Popen(cmd)))
    for src, p in procs:
        if p.wait() != 0:
            raise RuntimeError(f"nvcc failed on {src}")
    tmp = lib + f".tmp{os.getpid()}"
    subprocess.run([NVCC, "-shared", "-o", tmp] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"], check=True)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--debug" in sys.argv))
