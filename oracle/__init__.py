"""CPU oracle for the exact Euclidean distance transform -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper over ``edt_oracle.c`` (plain C, compiled with gcc).  Nothing here is part of the
product path: only the tests, the smoke check and the CPU-baseline leg of the benchmark may import it.
It shares no code with the CUDA library and never imports it.

The arithmetic lives in the C file, whose header states what is computed and how it is pinned
(paper, Section 2.1 "Distance transforms" for the definition, Section 2.3.2 for the separable form).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "edt_oracle.c")
_LIB = os.path.join(_HERE, "liboracle_edt.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over lines) if the library is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            p = ctypes.c_void_p
            common = [p, ctypes.c_int, p, p]
            lib.edt_oracle_brute.argtypes = common + [p, p, p, p]
            lib.edt_oracle_brute.restype = ctypes.c_int
            lib.edt_oracle_sep.argtypes = common + [p, p, p, p]
            lib.edt_oracle_sep.restype = ctypes.c_int
            lib.edt_oracle_sep_axes.argtypes = common + [p, ctypes.c_int, p, p, p, p]
            lib.edt_oracle_sep_axes.restype = ctypes.c_int
            lib.edt_oracle_threads.restype = ctypes.c_int
            lib.edt_oracle_set_threads.argtypes = [ctypes.c_int]
            _lib = lib
    return _lib


def threads() -> int:
    return int(_load().edt_oracle_threads())


def set_threads(t: int) -> None:
    _load().edt_oracle_set_threads(int(t))


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _run(kind, mask, sampling, want_idx, axes=None):
    """mask: (B, C, n_0..n_{d-1}) array, nonzero = foreground.  Returns a dict with
    ``dist`` float64, ``sqf`` float64, ``sq`` int64 (unit sampling only, else None) and
    ``idx`` int64 (B, C, ndim, n...) when asked for."""
    lib = _load()
    mask = np.ascontiguousarray(mask)
    if mask.dtype == np.bool_:
        mask = mask.view(np.uint8)
    if mask.dtype != np.uint8:
        raise TypeError("mask must be uint8 or bool")
    if mask.ndim < 3:
        raise ValueError("mask must be (B, C, spatial...)")
    ndim = mask.ndim - 2
    shape = np.asarray(mask.shape, dtype=np.int64)
    samp = None if sampling is None else np.ascontiguousarray(np.asarray(sampling, dtype=np.float64))
    if samp is not None and samp.shape != (ndim,):
        raise ValueError("sampling must have one entry per spatial axis")
    unit = samp is None or bool(np.all(samp == 1.0))
    dist = np.empty(mask.shape, dtype=np.float64)
    sqf = np.empty(mask.shape, dtype=np.float64)
    sq = np.empty(mask.shape, dtype=np.int64) if unit else None
    idx = np.empty(mask.shape[:2] + (ndim,) + mask.shape[2:], dtype=np.int64) if want_idx else None
    if kind == "brute":
        rc = lib.edt_oracle_brute(_ptr(mask), ndim, _ptr(shape), _ptr(samp), _ptr(dist), _ptr(sq), _ptr(sqf), _ptr(idx))
    else:
        ax = None if axes is None else np.ascontiguousarray(np.asarray(axes, dtype=np.int32))
        rc = lib.edt_oracle_sep_axes(
            _ptr(mask), ndim, _ptr(shape), _ptr(samp), _ptr(ax), 0 if ax is None else int(ax.size),
            _ptr(dist), _ptr(sq), _ptr(sqf), _ptr(idx),
        )
    if rc != 0:
        raise RuntimeError("edt oracle failed with status %d" % rc)
    return {"dist": dist, "sqf": sqf, "sq": sq, "idx": idx}


def brute(mask, sampling=None, want_idx=True):
    """The definition written out (every voxel against every background voxel). Tiny inputs only."""
    return _run("brute", mask, sampling, want_idx)


def sep(mask, sampling=None, want_idx=True):
    """Nested per-axis exhaustive minima over all axes: the parity authority."""
    return _run("sep", mask, sampling, want_idx)


def sep_axes(mask, axes, sampling=None, want_idx=True):
    """Intermediate after nested minima over the listed spatial axes only, in that order."""
    return _run("sep", mask, sampling, want_idx, axes=list(axes))


def virtual_background(mask, sampling=None, want_idx=True, kind="sep"):
    """The transform with the virtual out-of-bounds convention for images without background (paper,
    Section 2.3.2: the convention of scipy.ndimage): such an image is transformed as if it had exactly one
    background voxel, at coordinate -1 on spatial axis 0 and 0 on every other axis.

    Written as that definition: every image without background is extended by one slice in front of axis 0,
    foreground except for its voxel (0, .., 0); the extended image goes through the ordinary oracle, the extra
    slice is cut off again and the indices along axis 0 are shifted back by one.  Images with background are
    untouched.  Pins: the closed form and scipy.ndimage itself (tests/test_oracle_pins.py)."""
    run = brute if kind == "brute" else sep
    mask = np.ascontiguousarray(mask)
    res = run(mask, sampling, want_idx)
    ndim = mask.ndim - 2
    for b in range(mask.shape[0]):
        for c in range(mask.shape[1]):
            if not mask[b, c].all():
                continue
            ext = np.ones((1, 1, mask.shape[2] + 1) + mask.shape[3:], dtype=np.uint8)
            ext[(0, 0) + (0,) * ndim] = 0
            r = run(ext, sampling, want_idx)
            for key in ("dist", "sqf", "sq"):
                if res[key] is not None:
                    res[key][b, c] = r[key][0, 0, 1:]
            if want_idx:
                ix = r["idx"][0, 0][:, 1:].copy()
                ix[0] -= 1
                res["idx"][b, c] = ix
    return res
