"""Compile the CUDA library in-tree with nvcc for sm_100a.

    python -m paper_2407_04480_b200.build [--force] [--verbose]

Produces paper_2407_04480_b200/libloco_b200.so next to this file.  nvcc cross-compiles
without a GPU, so this runs anywhere the CUDA toolkit is installed.  The kernel templates are
instantiated in several object files (see csrc/loco_dispatch.h) that are compiled in parallel
and linked into the one shared library; the objects live in a temporary directory.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
import tempfile
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libloco_b200.so")
DEPS = [os.path.join(CSRC, f) for f in ("loco_api.cu", "loco_send_tu.cu", "loco_reduce_tu.cu", "loco_kernels.cuh",
                                        "loco_dispatch.h")] + [os.path.join(os.path.dirname(HERE), "include", "loco.h")]

NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC"]


def units():
    """(object name, source, extra defines) of every translation unit."""
    out = [("api", "loco_api.cu", [])]
    for g in (0, 1):
        for s in (0, 1, 2, 3):
            out.append(("send_g%d_s%d" % (g, s), "loco_send_tu.cu", ["-DLOCO_TU_GRAD=%d" % g, "-DLOCO_TU_STATE=%d" % s]))
    for o in (0, 1):
        for a in (0, 1):
            out.append(("reduce_o%d_a%d" % (o, a), "loco_reduce_tu.cu", ["-DLOCO_TU_OUT=%d" % o, "-DLOCO_TU_ADAM=%d" % a]))
    return out


def nvcc_path() -> str:
    p = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(p):
        raise RuntimeError("nvcc not found: the LoCo CUDA library cannot be built")
    return p


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(d) > t for d in DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not stale():
        return LIB
    nvcc = nvcc_path()
    extra = ["-Xptxas", "-v"] if verbose else []
    with tempfile.TemporaryDirectory(prefix="loco_build_") as tmpdir:
        def compile_one(u):
            name, src, defs = u
            obj = os.path.join(tmpdir, name + ".o")
            subprocess.check_call([nvcc, *NVCC_FLAGS, *extra, *defs, "-c", os.path.join(CSRC, src), "-o", obj])
            return obj

        with ThreadPoolExecutor(max_workers=max(1, os.cpu_count() or 1)) as ex:
            objs = list(ex.map(compile_one, units()))
        tmp = LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-cudart", "static",
                               "-Xcompiler", "-fPIC", "-o", tmp, *objs])
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
