"""Compile the CUDA sources under ``csrc/`` into ``libmxq.so`` next to this file (sm_100a only).

Run as ``python -m paper_2503_13565_b200.build`` or call :func:`build`.  nvcc cross-compiles,
so this works on a machine without a GPU.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libmxq.so")
OBJ = os.path.join(HERE, "build")
# the bounds-checked build (-DMXQ_DEBUG_BOUNDS: every plain global access of the linear kernels is tested against its
# buffer first; see csrc/mxq_device.cuh): a library of its own, loaded instead of the ordinary one when the environment
# has MXQ_LIBRARY=checked
LIB_CHECKED = os.path.join(HERE, "libmxq_checked.so")
OBJ_CHECKED = os.path.join(HERE, "build_checked")

NVCC_FLAGS = [
    "-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
]
# never --use_fast_math / -ftz=true: the smallest scale 2^-127 is an FP32 subnormal


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    lib, objdir = (LIB_CHECKED, OBJ_CHECKED) if checked else (LIB, OBJ)
    extra = ["-DMXQ_DEBUG_BOUNDS"] if checked else []
    srcs = sorted(glob.glob(os.path.join(CSRC, "*.cu")))
    hdrs = sorted(glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) +
                  glob.glob(os.path.join(HERE, "..", "include", "*.h")))
    os.makedirs(objdir, exist_ok=True)
    nvcc = _nvcc()
    jobs = []
    objs = []
    for s in srcs:
        o = os.path.join(objdir, os.path.basename(s)[:-3] + ".o")
        objs.append(o)
        if force or _stale(o, [s] + hdrs):
            cmd = [nvcc] + NVCC_FLAGS + extra + os.environ.get("MXQ_NVCC_FLAGS", "").split() + \
                (["-Xptxas", "-v"] if verbose else []) + ["-c", s, "-o", o]
            jobs.append(cmd)

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed: %s\n%s\n%s" % (" ".join(cmd), r.stdout, r.stderr))
        return r.stderr

    with ThreadPoolExecutor(max_workers=max(1, min(8, len(jobs)))) as ex:
        for out in ex.map(run, jobs):
            if verbose and out:
                sys.stderr.write(out)
    if force or jobs or _stale(lib, objs):
        tmp = lib + ".%d.tmp" % os.getpid()
        run([nvcc, "-shared", "-o", tmp] + objs + ["-Xcompiler", "-fvisibility=hidden"])
        os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
