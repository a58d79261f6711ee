"""Builds libprefixkv.so (sm_100a) next to this file with nvcc."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
LIB_PATH = os.path.join(_HERE, "libprefixkv.so")


def _sources():
    return sorted(glob.glob(os.path.join(_HERE, "csrc", "*.cu")))


def _headers():
    return sorted(glob.glob(os.path.join(_HERE, "csrc", "*.cuh"))) + \
        [os.path.join(_ROOT, "include", "prefixkv.h")]


def nvcc_path() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def is_stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(f) > t for f in _sources() + _headers())


def build_library(force: bool = False, verbose: bool = False) -> str:
    if not force and not is_stale():
        return LIB_PATH
    obj_dir = os.path.join(_HERE, "_build")
    os.makedirs(obj_dir, exist_ok=True)
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
             "-Xcompiler", "-fPIC", "-I", os.path.join(_ROOT, "include"),
             "-I", os.path.join(_HERE, "csrc")]
    if verbose:
        flags += ["-Xptxas", "-v"]
    objs, procs = [], []
    hdr_time = max(os.path.getmtime(f) for f in _headers())
    for src in _sources():
        obj = os.path.join(obj_dir, os.path.basename(src)[:-3] + ".o")
        objs.append(obj)
        if force or verbose or not os.path.exists(obj) or \
                os.path.getmtime(obj) < max(os.path.getmtime(src), hdr_time):
            procs.append((src, subprocess.Popen([nvcc_path(), *flags, "-c", src, "-o", obj])))
    for src, p in procs:
        if p.wait() != 0:
            raise RuntimeError("nvcc failed on " + src)
    tmp = LIB_PATH + ".%d.tmp" % os.getpid()
    subprocess.check_call([nvcc_path(), "-shared", "-o", tmp, *objs,
                           "-gencode", "arch=compute_100a,code=sm_100a"])
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
