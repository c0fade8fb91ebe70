"""Builds ``lib/libvmoba.so`` (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

``python -m paper_2506_23858_b200.build`` rebuilds; ``ensure_built()`` rebuilds only when a
source is newer than the library.  nvcc cross-compiles without a GPU.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB_DIR = os.path.join(HERE, "lib")
LIB_PATH = os.path.join(LIB_DIR, "libvmoba.so")
# the same library compiled with -DVMOBA_DEBUG: range-checked list indices and guarded workspace slices
DEBUG_LIB_PATH = os.path.join(LIB_DIR, "libvmoba_debug.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--extended-lambda", "-Xcompiler", "-fPIC", "-shared",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps():
    return sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(HERE, "..", "include", "*.h"))


def is_stale(debug: bool = False) -> bool:
    path = DEBUG_LIB_PATH if debug else LIB_PATH
    if not os.path.exists(path):
        return True
    t = os.path.getmtime(path)
    return any(os.path.getmtime(s) > t for s in _deps())


def build(verbose: bool = False, debug: bool = False) -> str:
    os.makedirs(LIB_DIR, exist_ok=True)
    nvcc = os.environ.get("NVCC", "nvcc")
    objs = []
    procs = []
    lib_path = DEBUG_LIB_PATH if debug else LIB_PATH
    for src in sources():
        obj = os.path.join(LIB_DIR, os.path.basename(src)[:-3] + (".debug.o" if debug else ".o"))
        cmd = [nvcc] + [f for f in NVCC_FLAGS if f != "-shared"] + (["-DVMOBA_DEBUG"] if debug else []) + ["-c", src, "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    for src, p in procs:
        out, _ = p.communicate()
        if verbose and out:
            print(out)
        if p.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}:\n{out}")
    tmp = lib_path + ".tmp"
    link = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", tmp] + objs
    r = subprocess.run(link, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{r.stdout}")
    os.replace(tmp, lib_path)
    return lib_path


def ensure_built(debug: bool = False) -> str:
    if is_stale(debug):
        build(debug=debug)
    return DEBUG_LIB_PATH if debug else LIB_PATH


if __name__ == "__main__":
    print(build(verbose="-v" in sys.argv, debug="--debug" in sys.argv))
