"""Build the shared libraries in-tree with nvcc for sm_100a.

libalsgd.so        the C-ABI library (include/alsgd.h)
libalsgd_dbg.so    the same sources compiled with -DALSGD_DEBUG_BOUNDS: every kernel access to an arena-owned
                   vector is range-checked, refused accesses are recorded and reported by alsgd_sync
libalsgd_sweep.so  the launch-shape benchmark library (include/alsgd_sweep.h)
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libalsgd.so")
LIB_DBG = os.path.join(HERE, "libalsgd_dbg.so")
LIB_SWEEP = os.path.join(HERE, "libalsgd_sweep.so")
SOURCES = ["alsgd_kernels.cu", "alsgd_ctx.cu", "alsgd_sched.cpp", "alsgd_static.cu"]
SWEEP_SOURCES = ["alsgd_sweep.cu"]
HEADERS = [os.path.join(CSRC, "alsgd_kernels.cuh"), os.path.join(CSRC, "alsgd_kernels_impl.cuh"),
           os.path.join(HERE, "..", "include", "alsgd.h"), os.path.join(HERE, "..", "include", "alsgd_sweep.h")]

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-lineinfo",
    "-gencode", "arch=compute_100a,code=sm_100a",
    # one IEEE operation per source operation: no multiply-add contraction, exact division and
    # square root, denormals kept (results must not depend on how the compiler schedules the math)
    "-fmad=false", "-prec-div=true", "-prec-sqrt=true", "-ftz=false",
    "-Xcompiler", "-fPIC,-ffp-contract=off,-fno-fast-math",
    "-shared",
]

TARGETS = {
    "main": (LIB, SOURCES, []),
    "debug": (LIB_DBG, SOURCES, ["-DALSGD_DEBUG_BOUNDS"]),
    "sweep": (LIB_SWEEP, SWEEP_SOURCES, []),
}


def needs_build(target: str = "main") -> bool:
    lib, sources, _ = TARGETS[target]
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, s) for s in sources] + HEADERS + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def _start(target: str, verbose: bool):
    lib, sources, extra = TARGETS[target]
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = lib + f".{os.getpid()}.tmp"
    cmd = [nvcc] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + [os.path.join(CSRC, s) for s in sources]
    return subprocess.Popen(cmd), tmp, lib, cmd


def build(force: bool = False, verbose: bool = False, targets=("main",)) -> str:
    """Compile the named targets (in parallel) if their sources are newer; returns the main library's path."""
    jobs = [_start(t, verbose) for t in targets if force or needs_build(t)]
    failed = None
    for proc, tmp, lib, cmd in jobs:
        if proc.wait() != 0:
            failed = failed or cmd
            continue
        os.replace(tmp, lib)
    if failed:
        raise subprocess.CalledProcessError(1, failed)
    return LIB


def build_all(force: bool = False, verbose: bool = False) -> str:
    return build(force, verbose, targets=tuple(TARGETS))


if __name__ == "__main__":
    names = [a for a in sys.argv[1:] if a in TARGETS] or (list(TARGETS) if "--all" in sys.argv else ["main"])
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, targets=tuple(names)))
