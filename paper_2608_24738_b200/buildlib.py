"""Builds the CUDA library in-tree with nvcc for sm_100a (no JIT cache, no other architecture).

Every ``csrc/*.cu`` is compiled to an object file under ``csrc/build/`` (recompiled only when it, or a header it
includes, changed) and the objects are linked into ``libtm_edt.so`` next to this file.
"""
from __future__ import annotations

import concurrent.futures
import glob
import os
import re
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ_DIR = os.path.join(CSRC, "build")
LIB = os.path.join(HERE, "libtm_edt.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")

COMPILE_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "-Xcompiler", "-fPIC,-fvisibility=hidden",
]
DEBUG_FLAGS = ["-DTM_EDT_DEBUG=1"]
LINK_FLAGS = ["-shared", "-cudart", "static", "-gencode", "arch=compute_100a,code=sm_100a"]

_INCLUDE = re.compile(r'^\s*#\s*include\s+"([^"]+)"', re.M)


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps(path, seen=None):
    """The file and every header it includes with quotes, recursively."""
    seen = set() if seen is None else seen
    path = os.path.normpath(path)
    if path in seen or not os.path.exists(path):
        return seen
    seen.add(path)
    with open(path) as fh:
        text = fh.read()
    for inc in _INCLUDE.findall(text):
        _deps(os.path.join(os.path.dirname(path), inc), seen)
    return seen


def _newer(target, deps):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def lib_path(debug: bool = False) -> str:
    return LIB if not debug else os.path.join(HERE, "libtm_edt_debug.so")


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compile csrc/*.cu and link libtm_edt.so next to this file; returns its path.

    debug=True builds libtm_edt_debug.so with -DTM_EDT_DEBUG=1: the kernels check their shared-memory and
    global-memory indices and report a violation through the call's status instead of touching the address."""
    out = lib_path(debug)
    all_deps = set().union(*[_deps(src) for src in sources()]) | {os.path.abspath(__file__)}
    if not force and not verbose and not _newer(out, all_deps):
        return out  # up to date (object files need not exist: a copy of the tree carries the library alone)
    os.makedirs(OBJ_DIR, exist_ok=True)
    suffix = ".debug.o" if debug else ".o"
    flags = COMPILE_FLAGS + (DEBUG_FLAGS if debug else []) + (["-Xptxas", "-v"] if verbose else [])
    jobs = []
    objs = []
    for src in sources():
        obj = os.path.join(OBJ_DIR, os.path.basename(src)[:-3] + suffix)
        objs.append(obj)
        if force or _newer(obj, _deps(src) | {os.path.abspath(__file__)}):
            jobs.append([NVCC] + flags + ["-c", src, "-o", obj])
    if jobs:
        with concurrent.futures.ThreadPoolExecutor(max_workers=max(1, min(len(jobs), os.cpu_count() or 1))) as pool:
            for rc in pool.map(subprocess.call, jobs):
                if rc != 0:
                    raise RuntimeError("nvcc failed")
    if jobs or _newer(out, objs):
        tmp = out + ".tmp.%d" % os.getpid()
        subprocess.check_call([NVCC] + LINK_FLAGS + ["-o", tmp] + objs)
        os.replace(tmp, out)
    return out


if __name__ == "__main__":
    import sys

    print(build(force="-f" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
