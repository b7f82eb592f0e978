"""Builds the CUDA library ``libdq.so`` in-tree with nvcc for sm_100a.

Usage: ``python -m paper_2107_14575_b200.build [--force] [--verbose] [--checked]``
Objects go to ``paper_2107_14575_b200/_build``; the shared library sits next
to the Python binding so that it travels with the source tree.

``--checked`` builds ``libdq_checked.so`` instead (objects in ``_build_checked``): the same
sources with ``-DDQ_CHECKED``, under which every store of a kernel to global memory checks that
it lies inside the buffer it belongs to and raises ``DQ_STAT_INTERNAL`` instead of storing if it
does not.  ``DQ_LIBRARY=<path>`` makes the Python binding load that library.
"""
from __future__ import annotations

import concurrent.futures as cf
import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
OBJ = os.path.join(PKG, "_build")
LIB = os.path.join(PKG, "libdq.so")

SOURCES = ["dq_layout.cu", "dq_tma.cu", "dq_norms.cu", "dq_bits.cu", "dq_quantize.cu", "dq_fused.cu", "dq_unpack.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def _deps_mtime() -> float:
    paths = [os.path.join(ROOT, "include", "dq.h")]
    paths += [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    return max(os.path.getmtime(p) for p in paths)


LIB_CHECKED = os.path.join(PKG, "libdq_checked.so")


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    LIB = LIB_CHECKED if checked else globals()["LIB"]
    OBJ = globals()["OBJ"] + ("_checked" if checked else "")
    newest = _deps_mtime()
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= newest:
        return LIB
    os.makedirs(OBJ, exist_ok=True)
    nvcc = _nvcc()
    extra = (["-Xptxas", "-v"] if verbose else []) + (["-DDQ_CHECKED"] if checked else [])

    def compile_one(src: str) -> str:
        obj = os.path.join(OBJ, src.replace(".cu", ".o"))
        if not force and os.path.exists(obj) and os.path.getmtime(obj) >= newest:
            return obj
        cmd = [nvcc, *NVCC_FLAGS, *extra, "-c", os.path.join(CSRC, src), "-o", obj]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or r.returncode != 0:
            sys.stderr.write("$ " + " ".join(cmd) + "\n" + r.stdout + r.stderr)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed on " + src)
        return obj

    with cf.ThreadPoolExecutor(max_workers=min(8, len(SOURCES))) as ex:
        objs = list(ex.map(compile_one, SOURCES))
    tmp = LIB + ".tmp.%d" % os.getpid()
    cmd = [nvcc, "-shared", "-o", tmp, *objs, "-gencode", "arch=compute_100a,code=sm_100a",
           "-cudart", "static"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
        raise RuntimeError("link failed")
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, checked="--checked" in sys.argv))
