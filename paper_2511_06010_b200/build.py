"""Builds csrc/libmoska.so for sm_100a with nvcc (cross-compiles without a GPU).

Every .cu file is compiled to an object of its own (in parallel, only when it or a header is
newer than the object) under csrc/_build/, then linked.  Run as
`python -m paper_2511_06010_b200.build [--force] [-v] [--debug]` or call `build()`.
`--debug` / `build(debug=True)` builds csrc/libmoska_debug.so instead: the same sources with
-DMOSKA_DEBUG_GUARDS (guard words around the workspace regions, capacity checks on the work lists).
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ_DIR = os.path.join(CSRC, "_build")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(CSRC, "libmoska.so")
LIB_DEBUG = os.path.join(CSRC, "libmoska_debug.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _headers():
    return glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(INCLUDE, "*.h"))


def _newer(deps, target) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(p) > t for p in deps)


def _stale(lib: str = LIB) -> bool:
    return _newer(sources() + _headers(), lib)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    lib = LIB_DEBUG if debug else LIB
    if not force and not _stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ_DIR, exist_ok=True)
    headers = _headers()
    extra = ["-DMOSKA_DEBUG_GUARDS"] if debug else []
    suffix = ".debug.o" if debug else ".o"
    jobs = []
    objects = []
    for src in sources():
        obj = os.path.join(OBJ_DIR, os.path.basename(src)[:-3] + suffix)
        objects.append(obj)
        if force or _newer([src] + headers, obj):
            cmd = [nvcc, *NVCC_FLAGS, *extra, "-I", INCLUDE, "-I", CSRC, "-c", src, "-o", obj]
            if verbose:
                cmd[1:1] = ["-Xptxas", "-v"]
            jobs.append(cmd)
    with ThreadPoolExecutor(max_workers=min(8, max(1, len(jobs)))) as pool:
        results = list(pool.map(lambda c: subprocess.run(c, capture_output=True, text=True), jobs))
    for cmd, r in zip(jobs, results):
        if verbose or r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
        if r.returncode != 0:
            raise subprocess.CalledProcessError(r.returncode, cmd)
    known = {os.path.basename(s)[:-3] for s in sources()}
    for name in os.listdir(OBJ_DIR):  # objects of source files that no longer exist
        if name.split(".")[0] not in known:
            os.remove(os.path.join(OBJ_DIR, name))
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared",
                           "-o", lib, *objects])
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
