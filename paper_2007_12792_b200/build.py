"""Builds ``libdn.so`` (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

    python -m paper_2007_12792_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdn.so")
# (source, object name, extra flags): the 3D strip kernel is compiled in two parts (its template instantiations for
# m <= 4 and for m >= 5), which run side by side
SOURCES = [(f, f.replace(".cu", ".o"), []) for f in
           ["dn_api.cu", "dn_aux.cu", "dn_generic.cu", "dn_tiled2d.cu", "dn_strip2d.cu", "dn_row2d.cu", "dn_tiled3d.cu",
            "dn_strip3d.cu", "dn_static.cu", "dn_burgers.cu", "dn_cg.cu"]]
SOURCES.append(("dn_strip3d.cu", "dn_strip3d_hi.o", ["-DDN_S3_PART=1"]))
HEADERS = [os.path.join(CSRC, "dn_internal.cuh"), os.path.join(ROOT, "include", "dn.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I" + os.path.join(ROOT, "include"), "-I" + CSRC]


def _stale(target, deps):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    nvcc = os.environ.get("NVCC", "nvcc")
    objdir = os.path.join(HERE, "_build")
    os.makedirs(objdir, exist_ok=True)
    objs = []
    procs = []
    for src, objname, extra in SOURCES:
        path = os.path.join(CSRC, src)
        obj = os.path.join(objdir, objname)
        objs.append(obj)
        if force or _stale(obj, [path] + HEADERS):
            cmd = [nvcc] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-c", path, "-o", obj]
            procs.append((objname, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    failed = False
    for src, p in procs:
        out, _ = p.communicate()
        if p.returncode != 0 or verbose:
            sys.stderr.write(f"--- {src}\n{out}\n")
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    if force or procs or _stale(LIB, objs):
        subprocess.run([nvcc, "-shared", "-o", LIB] + objs + ["-lcudart"], check=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
