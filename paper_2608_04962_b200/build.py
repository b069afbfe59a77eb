"""Builds ``libspecroll.so`` (the C-ABI library of sm_100a kernels) in-tree with nvcc."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libspecroll.so")
LIB_CHECK = os.path.join(HERE, "libspecroll_check.so")   # the same library with the kernels' index checks compiled in
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
         "-Xcompiler", "-fPIC"]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale(lib=LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        glob.glob(os.path.join(HERE, "..", "include", "*.h"))
    return any(os.path.getmtime(p) > t for p in deps)


def build(force: bool = False, verbose: bool = False, check: bool = False) -> str:
    """Compile every kernel for sm_100a and link the shared library.  Returns its path.
    check=True builds the debug variant (-DSPECROLL_CHECK: index checks in the kernels) beside it."""
    lib = LIB_CHECK if check else LIB
    if not force and not _stale(lib):
        return lib
    objs = []
    procs = []
    bdir = "build_check" if check else "build"
    os.makedirs(os.path.join(HERE, bdir), exist_ok=True)
    flags = list(FLAGS) + os.environ.get("SPECROLL_NVCC_FLAGS", "").split() + (["-DSPECROLL_CHECK"] if check else [])
    if verbose:
        flags = flags + ["-Xptxas", "-v"]
    for src in sources():
        obj = os.path.join(HERE, bdir, os.path.basename(src)[:-3] + ".o")
        objs.append(obj)
        procs.append((src, subprocess.Popen([NVCC, *flags, "-c", src, "-o", obj],
                                            stdout=subprocess.PIPE, stderr=subprocess.STDOUT)))
    failed = False
    for src, p in procs:
        out = p.communicate()[0].decode()
        if p.returncode != 0 or verbose:
            sys.stderr.write(f"--- {os.path.basename(src)}\n{out}\n")
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    tmp = lib + f".tmp{os.getpid()}"
    subprocess.check_call([NVCC, "-shared", "-o", tmp, *objs])
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, check="--check" in sys.argv))
