"""Builds the C-ABI CUDA library in-tree: paper_2607_27042_b200/libgptq2d.so (sm_100a only)."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libgptq2d.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
         "-Xcompiler", "-fPIC", "--fmad=true"]


def sources():
    return sorted(f for f in os.listdir(CSRC) if f.endswith(".cu"))


def _newest_header():
    t = 0.0
    for root in (CSRC, os.path.join(os.path.dirname(HERE), "include")):
        for f in os.listdir(root):
            if f.endswith((".cuh", ".h")):
                t = max(t, os.path.getmtime(os.path.join(root, f)))
    return t


LIB_CHECKED = os.path.join(HERE, "libgptq2d_checked.so")


LIB_STATS = os.path.join(HERE, "libgptq2d_stats.so")


def build(force=False, verbose=False, checked=False, stats=False):
    """checked=True builds libgptq2d_checked.so: the same library with -DGPTQ2D_CHECKED, in which every index
    that feeds a shared- or global-memory access of the sweep kernels is range-checked and a violation is
    reported through the call's status words (nothing traps).  Test use only: it is slow."""
    # stats=True builds libgptq2d_stats.so: in-kernel cycle counters of the sweep kernels (-DTILED_STATS
    # -DFUSED_STATS), printed by a few CTAs at the end of a launch.  Measurement aid, not a product build.
    obj_dir = OBJ + ("_checked" if checked else "_stats" if stats else "")
    lib = LIB_CHECKED if checked else LIB_STATS if stats else LIB
    extra = ["-DGPTQ2D_CHECKED"] if checked else ["-DTILED_STATS", "-DFUSED_STATS"] if stats else []
    os.makedirs(obj_dir, exist_ok=True)
    hdr = _newest_header()
    jobs = []
    for src in sources():
        s = os.path.join(CSRC, src)
        o = os.path.join(obj_dir, src[:-3] + ".o")
        if force or not os.path.exists(o) or os.path.getmtime(o) < max(os.path.getmtime(s), hdr):
            cmd = [NVCC] + FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-c", s, "-o", o]
            jobs.append(cmd)

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed: " + " ".join(cmd))

    with ThreadPoolExecutor(max_workers=4) as ex:
        list(ex.map(run, jobs))
    objs = [os.path.join(obj_dir, s[:-3] + ".o") for s in sources()]
    if jobs or not os.path.exists(lib):
        subprocess.check_call([NVCC, "-arch=sm_100a", "-shared", "-o", lib] + objs + ["-lcudart"])
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv,
                stats="--stats" in sys.argv))
