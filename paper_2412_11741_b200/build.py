"""Builds libcsr.so (the C-ABI library) in-tree with nvcc for sm_100a.

Every .cu file under csrc/ is compiled to an object of its own (in parallel, only when it
or a header is newer than its object) and the objects are linked into libcsr.so.

`python -m paper_2412_11741_b200.build --debug` builds libcsr_debug.so instead: the same
library compiled with -DCSR_DEBUG_CHECKS, whose kernels record every index they had to clamp
before a gather (csr_device_status then reports CSR_ERR_BOUNDS).  Load it by setting
CSR_LIBRARY_PATH to its path before importing the package.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
OBJ = os.path.join(PKG, "_build")
LIB = os.path.join(PKG, "libcsr.so")
OBJ_DEBUG = os.path.join(PKG, "_build_debug")
LIB_DEBUG = os.path.join(PKG, "libcsr_debug.so")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _sources():
    return sorted(f for f in os.listdir(CSRC) if f.endswith(".cu"))


def _headers():
    return [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cuh")] + [os.path.join(ROOT, "include", "csr.h")]


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def needs_build(debug: bool = False) -> bool:
    return _stale(LIB_DEBUG if debug else LIB, [os.path.join(CSRC, f) for f in _sources()] + _headers())


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    lib, objdir = (LIB_DEBUG, OBJ_DEBUG) if debug else (LIB, OBJ)
    if not force and not needs_build(debug):
        return lib
    os.makedirs(objdir, exist_ok=True)
    nvcc, hdrs = _nvcc(), _headers()
    flags = FLAGS + (["-DCSR_DEBUG_CHECKS"] if debug else [])

    def compile_one(src: str):
        obj = os.path.join(objdir, src[:-3] + ".o")
        if not force and not _stale(obj, [os.path.join(CSRC, src)] + hdrs):
            return obj, 0, ""
        cmd = [nvcc] + flags + (["-Xptxas=-v"] if verbose else []) + ["-I", os.path.join(ROOT, "include"), "-I", CSRC, "-c",
                                                                        os.path.join(CSRC, src), "-o", obj]
        res = subprocess.run(cmd, capture_output=True, text=True)
        return obj, res.returncode, res.stdout + res.stderr

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        results = list(pool.map(compile_one, _sources()))
    for _, rc, log in results:
        if verbose or rc != 0:
            sys.stderr.write(log)
    if any(rc != 0 for _, rc, _ in results):
        raise RuntimeError("nvcc failed building libcsr.so")
    res = subprocess.run([nvcc, "-shared", "-o", lib] + [o for o, _, _ in results] + ["-lcudart"], capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("linking the library failed")
    return lib


if __name__ == "__main__":
    print(build(force="-f" in sys.argv or "-v" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
