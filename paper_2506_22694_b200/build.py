"""Builds libvocabtrim.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

Usage: python -m paper_2506_22694_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libvocabtrim.so")
OBJ_DIR = os.path.join(HERE, "_build")
LIB_STAMPS = os.path.join(HERE, "libvocabtrim_stamps.so")     # -DVT_STAMPS: phase stamps in the head kernel
OBJ_DIR_STAMPS = os.path.join(HERE, "_build_stamps")

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-lineinfo",
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-Xcompiler", "-fPIC",
    "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]


def _sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps():
    return _sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(p) > t for p in _deps())


def build(force: bool = False, verbose: bool = False, stamps: bool = False) -> str:
    """Compile every .cu under csrc/ (one object each, in parallel) and link the shared library.
    stamps=True builds the instrumented twin (libvocabtrim_stamps.so, -DVT_STAMPS) instead."""
    LIB, OBJ_DIR = (LIB_STAMPS, OBJ_DIR_STAMPS) if stamps else (globals()["LIB"], globals()["OBJ_DIR"])
    if not force and not needs_build(LIB):
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    os.makedirs(OBJ_DIR, exist_ok=True)
    extra = (["-Xptxas", "-v"] if verbose else []) + (["-DVT_STAMPS"] if stamps else [])
    procs, objs = [], []
    hdr_time = max(os.path.getmtime(p) for p in _deps() if not p.endswith(".cu"))
    for src in _sources():
        obj = os.path.join(OBJ_DIR, os.path.basename(src)[:-3] + ".o")
        objs.append(obj)
        if (not force and os.path.exists(obj) and os.path.getmtime(obj) > os.path.getmtime(src)
                and os.path.getmtime(obj) > hdr_time):
            continue
        cmd = [nvcc] + NVCC_FLAGS + extra + ["-c", src, "-o", obj]
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    failed = False
    for src, p in procs:
        out, _ = p.communicate()
        if p.returncode != 0 or verbose:
            sys.stderr.write("== %s\n%s\n" % (os.path.basename(src), out))
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    tmp = LIB + ".%d.tmp" % os.getpid()
    subprocess.check_call([nvcc, "-shared", "-o", tmp] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"])
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, stamps="--stamps" in sys.argv))
