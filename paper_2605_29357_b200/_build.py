"""Builds libpn.so (the C-ABI library) in-tree with nvcc for sm_100a.

Objects are cached under csrc/_build/ and rebuilt when a source or header is newer.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
OBJ = os.path.join(CSRC, "_build")
LIB = os.path.join(HERE, "libpn.so")
SOURCES = ["kernels.cu", "no_alloc.cu", "probe.cu", "lower.cpp", "lower_col.cpp", "descriptor.cpp", "spec.cpp", "api.cpp", "sequence.cpp"]
HEADERS = [os.path.join(CSRC, "plan.h"), os.path.join(CSRC, "graph.h"), os.path.join(CSRC, "spec.h"), os.path.join(CSRC, "handle.h"), os.path.join(CSRC, "lower_common.h"),
           os.path.join(CSRC, "device_lib.cuh"), os.path.join(INCLUDE, "pn.h")]
INSTANCES = [(1, 8, 4), (4, 2, 4), (4, 4, 2), (8, 1, 4), (8, 2, 2)]   # (VL, NG, K), as listed in kernels.cu
FLAGS = ["-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
         "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden"]


def _nvcc() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the CUDA toolkit is needed to build libpn.so")


def _embed_device_source() -> None:
    """plan.h + device_lib.cuh as one C++ raw string literal: the text that the kernels
    specialised at run time are compiled from."""
    text = ""
    for name in ("plan.h", "device_lib.cuh"):
        with open(os.path.join(CSRC, name)) as f:
            text += "".join(line for line in f if not line.startswith("#pragma once"))
    assert ')PNSRC"' not in text
    out = os.path.join(OBJ, "device_src.inc")
    new = 'R"PNSRC(' + text + ')PNSRC"\n'
    if not os.path.exists(out) or open(out).read() != new:
        with open(out, "w") as f:
            f.write(new)


def build_library(force: bool = False, verbose: bool = False) -> str:
    os.makedirs(OBJ, exist_ok=True)
    _embed_device_source()
    nvcc = _nvcc()
    newest_header = max(os.path.getmtime(h) for h in HEADERS)
    objs, relink = [], force or not os.path.exists(LIB)
    jobs = []
    units = [(src, src + ".o", []) for src in SOURCES]
    # the interpreter kernels: one translation unit per tile shape, so that they build side by side
    units += [("kernels.cu", "kernels_%d_%d_%d.o" % inst, ["-DPN_VL=%d" % inst[0], "-DPN_NG=%d" % inst[1], "-DPN_K=%d" % inst[2]])
              for inst in INSTANCES]
    for src, obj, defs in units:
        s = os.path.join(CSRC, src)
        o = os.path.join(OBJ, obj)
        objs.append(o)
        if force or not os.path.exists(o) or os.path.getmtime(o) < max(os.path.getmtime(s), newest_header):
            jobs.append([nvcc, "-c", *FLAGS, *defs, "-o", o, s])
    if jobs:   # the translation units are independent: compile them side by side
        from concurrent.futures import ThreadPoolExecutor

        def run(cmd):
            if verbose:
                print(" ".join(cmd), file=sys.stderr)
            subprocess.run(cmd, check=True)

        with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 1)) as pool:
            list(pool.map(run, jobs))
        relink = True
    if relink or any(os.path.getmtime(o) > os.path.getmtime(LIB) for o in objs):
        subprocess.run([nvcc, "-shared", "-o", LIB, *objs], check=True)
    return LIB


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose=True))
