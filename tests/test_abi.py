"""The C-ABI library loads, exports every symbol the header declares, and rejects bad arguments
before doing any device work (these checks need no GPU)."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2608_24738_b200 import binding, buildlib

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    buildlib.build()
    return binding.lib()


def test_header_symbols_are_exported(L):
    header = open(os.path.join(ROOT, "include", "tm_edt.h")).read() + open(os.path.join(ROOT, "include", "tm_morph.h")).read() + open(os.path.join(ROOT, "include", "tm_cdt.h")).read()
    declared = set(re.findall(r"TM_EDT_API[^;(]*?\b(tm_\w+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name


def test_version_and_strerror(L):
    assert "sm_100a" in binding.tm_edt_version()
    texts = [binding.tm_edt_strerror(s) for s in range(8)]  # TM_EDT_OK .. TM_EDT_ERR_DEBUG_CHECK
    assert all(texts) and "unknown status" not in texts and len(set(texts)) == 8
    assert not binding.tm_edt_debug_build() and binding.tm_edt_debug_last_violation()[0] == 0
    assert "tm_edt_noalloc" in binding.tm_edt_strerror(binding.ERR_TOO_LARGE)
    assert binding.tm_edt_strerror(99) == "unknown status"


def _call(L, inp=1, ndim=2, shape=(1, 1, 4, 4), sampling=None, d=1, s=0, x=0):
    shp = (ctypes.c_int64 * len(shape))(*shape) if shape is not None else None
    smp = (ctypes.c_double * len(sampling))(*sampling) if sampling is not None else None
    fake = lambda v: ctypes.c_void_p(0x1000 * v) if v else None  # never dereferenced on these paths
    return L.tm_edt(fake(inp), ndim, shp, smp, fake(2 * d), fake(3 * s), fake(4 * x), None)


def test_invalid_arguments_return_before_any_device_work(L):
    E = binding
    assert _call(L, inp=0) == E.ERR_INVALID_ARG
    assert _call(L, shape=None) == E.ERR_INVALID_ARG
    assert _call(L, ndim=0, shape=(1, 1)) == E.ERR_INVALID_ARG
    assert _call(L, ndim=9, shape=(1, 1) + (2,) * 9) == E.ERR_INVALID_ARG
    assert _call(L, shape=(1, 1, -1, 4)) == E.ERR_INVALID_ARG
    assert _call(L, shape=(-1, 1, 4, 4)) == E.ERR_INVALID_ARG
    assert _call(L, sampling=(1.0, 0.0)) == E.ERR_INVALID_ARG
    assert _call(L, sampling=(1.0, -2.0)) == E.ERR_INVALID_ARG
    assert _call(L, sampling=(float("nan"), 1.0)) == E.ERR_INVALID_ARG
    assert _call(L, sampling=(float("inf"), 1.0)) == E.ERR_INVALID_ARG
    assert _call(L, d=0, s=0, x=0) == E.ERR_INVALID_ARG


def test_flag_word_of_tm_edt_ex(L):
    """Unknown flag bits are an argument error; with the flat-index flag the index buffer is one int64 per voxel,
    which changes the overlap rule between the outputs."""
    shp = (ctypes.c_int64 * 4)(1, 1, 4, 4)
    inp, d = ctypes.c_void_p(0x20000), ctypes.c_void_p(0x10000)
    assert L.tm_edt_ex(inp, 2, shp, None, None, d, None, None, 8, None, 0, None) == binding.ERR_INVALID_ARG
    assert L.tm_edt_ex(inp, 2, shp, None, None, d, None, None, 0x80000000, None, 0, None) == binding.ERR_INVALID_ARG
    x = ctypes.c_void_p(0x30000)          # 16 voxels: 256 B of coordinate planes, 128 B of flat indices
    after = ctypes.c_void_p(0x30000 + 128)  # inside the coordinate planes, just behind the flat indices
    assert L.tm_edt_ex(inp, 2, shp, None, None, after, None, x, 0, None, 0, None) == binding.ERR_INVALID_ARG
    assert L.tm_edt_ex(inp, 2, shp, None, None, after, None, x, binding.FLAG_FLAT_INDEX, None, 0, None) == binding.ERR_BAD_POINTER
    # float64 distances: 8-byte alignment and 8 bytes per voxel in the overlap rule
    assert L.tm_edt_ex(inp, 2, shp, None, None, ctypes.c_void_p(0x10004), None, None, binding.FLAG_DIST_F64, None, 0,
                       None) == binding.ERR_INVALID_ARG
    sq = ctypes.c_void_p(0x10000 + 64)   # behind 16 float32 distances, inside 16 float64 ones
    assert L.tm_edt_ex(inp, 2, shp, None, None, d, sq, None, 0, None, 0, None) == binding.ERR_BAD_POINTER
    assert L.tm_edt_ex(inp, 2, shp, None, None, d, sq, None, binding.FLAG_DIST_F64, None, 0, None) == binding.ERR_INVALID_ARG
    # strides: negative ones are rejected; a strided mask must not reach into an output
    bad = (ctypes.c_int64 * 4)(16, 16, -4, 1)
    assert L.tm_edt_ex(inp, 2, shp, bad, None, d, None, None, 0, None, 0, None) == binding.ERR_INVALID_ARG
    wide = (ctypes.c_int64 * 4)(0, 0, 0x4000, 1)  # rows 16 KiB apart: the mask spans 48 KiB + 4 bytes
    assert L.tm_edt_ex(ctypes.c_void_p(0x8000), 2, shp, wide, None, d, None, None, 0, None, 0, None) == binding.ERR_INVALID_ARG


def test_workspace_bytes_of_tm_edt_ex(L):
    base = binding.tm_edt_workspace_bytes((2, 1, 64, 64, 64))
    n = 2 * 64 ** 3
    assert binding.tm_edt_ex_workspace_bytes((2, 1, 64, 64, 64)) == base
    strides = (64 ** 3 * 2, 64 ** 3 * 2, 64 * 64 * 2, 64 * 2, 2)  # every second byte of a larger buffer
    assert binding.tm_edt_ex_workspace_bytes((2, 1, 64, 64, 64), strides) >= base + n
    f64 = binding.tm_edt_ex_workspace_bytes((2, 1, 64, 64, 64), None, binding.FLAG_DIST_F64)
    assert f64 >= base + 8 * n
    assert binding.tm_edt_ex_workspace_bytes((2, 1, 64, 64, 64), None, binding.FLAG_DIST_F64, with_indices=True) == base
    with pytest.raises(binding.TmEdtError):
        binding.tm_edt_ex_workspace_bytes((1, 1, 4, 4), (16, 16, -4, 1))


def test_unsupported(L):
    E = binding
    assert _call(L, shape=(1, 1, E.MAX_EXTENT + 1, 4)) == E.ERR_UNSUPPORTED
    assert _call(L, sampling=(1.0, 2.0), s=1) == E.ERR_UNSUPPORTED
    assert _call(L, shape=(1, 1, 8192, 8192, 64), ndim=3) == E.ERR_UNSUPPORTED  # > 2^31 - 1 voxels per image
    assert _call(L, shape=(1 << 20, 1 << 10, 8192, 8192), ndim=2) == E.ERR_UNSUPPORTED  # > 2^40 elements


def test_empty_problem_is_ok_without_touching_pointers(L):
    assert _call(L, shape=(0, 1, 4, 4)) == binding.OK
    assert _call(L, shape=(1, 1, 4, 0)) == binding.OK
    assert binding.tm_edt_last_launch_count() == 0


def test_overlapping_buffers_are_rejected(L):
    shp = (ctypes.c_int64 * 4)(1, 1, 4, 4)
    a = ctypes.c_void_p(0x10000)
    b = ctypes.c_void_p(0x10008)  # overlaps a 64-byte float output starting at 0x10000
    assert L.tm_edt(a, 2, shp, None, b, None, None, None) == binding.ERR_INVALID_ARG
    assert L.tm_edt(ctypes.c_void_p(0x20000), 2, shp, None, a, b, None, None) == binding.ERR_INVALID_ARG


def test_misaligned_outputs_are_rejected(L):
    shp = (ctypes.c_int64 * 4)(1, 1, 4, 4)
    inp = ctypes.c_void_p(0x20000)
    assert L.tm_edt(inp, 2, shp, None, ctypes.c_void_p(0x10002), None, None, None) == binding.ERR_INVALID_ARG
    assert L.tm_edt(inp, 2, shp, None, None, ctypes.c_void_p(0x10004), None, None) == binding.ERR_INVALID_ARG
    assert L.tm_edt(inp, 2, shp, None, None, None, ctypes.c_void_p(0x10004), None) == binding.ERR_INVALID_ARG


def test_host_memory_is_not_accepted_as_device_memory(L):
    # Valid arguments, but the buffers are ordinary host arrays: BAD_POINTER (with or without a GPU present).
    m = np.ones((1, 1, 4, 4), dtype=np.uint8)
    out = np.zeros((1, 1, 4, 4), dtype=np.float32)
    shp = (ctypes.c_int64 * 4)(1, 1, 4, 4)
    rc = L.tm_edt(m.ctypes.data_as(ctypes.c_void_p), 2, shp, None, out.ctypes.data_as(ctypes.c_void_p), None, None, None)
    assert rc == binding.ERR_BAD_POINTER


def test_workspace_bytes(L):
    assert binding.tm_edt_workspace_bytes((1, 1, 0, 4)) == 0
    assert binding.tm_edt_workspace_bytes((1, 1, 64)) == 0  # a single pass needs no scratch
    assert binding.tm_edt_workspace_bytes((2, 3, 64, 64)) == 0  # first two axes are fused in one kernel
    assert binding.tm_edt_workspace_bytes((2, 3, 64, 64, 64)) >= 2 * (2 * 3 * 64 ** 3)  # 2-byte entries
    assert binding.tm_edt_workspace_bytes((1, 1, 300, 300)) >= 2 * 300 * 300  # generic path: 16-bit offset planes
    assert binding.tm_edt_workspace_bytes((1, 1, 1024, 1024)) == 6 * 1024 * 1024  # wide path, two axes: key + offset
    assert binding.tm_edt_workspace_bytes((1, 1, 256, 256, 256)) == 14 * 256 ** 3  # three axes: 2 keys + 1 + 2 offsets
    # one particular call: without an index output no offsets are carried
    assert binding.tm_edt_workspace_bytes_for((1, 1, 256, 256, 256), want_indices=True) == 14 * 256 ** 3
    assert binding.tm_edt_workspace_bytes_for((1, 1, 256, 256, 256), want_indices=False) == 8 * 256 ** 3
    assert binding.tm_edt_workspace_bytes_for((1, 1, 1024, 1024), want_indices=False) == 4 * 1024 * 1024
    assert binding.tm_edt_workspace_bytes_for((2, 1, 128, 128, 128), (2.5, 0.8, 1.0)) == 4 * 2 * 128 ** 3


def test_workspace_bytes_cover_every_sampling(L):
    """tm_edt_workspace_bytes(shape) suffices whatever the sampling: the planner may choose another kernel family
    for non-unit sampling (shapes on both sides of the limit up to which integer keys fit 31 bits), and a call with a
    workspace of the reported size must never be refused as too small.  No GPU: the call stops at the pointer check,
    which comes after the size check."""
    shapes = [(1, 1, 2, 66, 1024, 1024), (1, 1, 2, 60, 520, 516), (1, 1, 4, 4, 600, 600), (1, 1, 900, 900, 8),
              (1, 1, 1024, 1024), (1, 1, 300, 300, 300), (2, 1, 128, 128, 128), (1, 1, 16, 128, 128, 128),
              (1, 1, 5, 200, 40, 520)]
    for shape in shapes:
        ndim = len(shape) - 2
        need = binding.tm_edt_workspace_bytes(shape)
        shp = (ctypes.c_int64 * len(shape))(*shape)
        for sampling in (None, tuple(1.0 + 0.37 * k for k in range(ndim)), (2.5,) * ndim):
            smp = (ctypes.c_double * ndim)(*sampling) if sampling is not None else None
            assert binding.tm_edt_workspace_bytes_for(shape, sampling, want_indices=True) <= need
            fake = lambda v: ctypes.c_void_p((v << 42) + 4096)  # far apart (no overlap), never dereferenced: the pointer check refuses them
            rc = L.tm_edt_ws(fake(1), ndim, shp, smp, fake(2), None, fake(3), fake(4), ctypes.c_size_t(need), None)
            assert rc == binding.ERR_BAD_POINTER, (shape, sampling, rc)
            if need > 0:
                rc = L.tm_edt_ws(fake(1), ndim, shp, smp, fake(2), None, fake(3), fake(4),
                                 ctypes.c_size_t(binding.tm_edt_workspace_bytes_for(shape, sampling, want_indices=True) - 1), None)
                assert rc == binding.ERR_ALLOC or binding.tm_edt_workspace_bytes_for(shape, sampling, want_indices=True) == 0
    with pytest.raises(binding.TmEdtError):
        binding.tm_edt_workspace_bytes((1, 1, binding.MAX_EXTENT + 1))


def test_binding_refuses_host_tensor():
    import torch

    with pytest.raises(ValueError):
        binding.tm_edt(torch.ones((1, 1, 4, 4), dtype=torch.uint8))


def test_morphology_argument_errors(L):
    """tm_grey_morph / tm_binary_morph reject bad arguments before any device work."""
    E = binding
    shp = (ctypes.c_int64 * 4)(1, 1, 8, 8)
    fps = (ctypes.c_int64 * 2)(3, 3)
    fp = (ctypes.c_uint8 * 9)(*([1] * 9))
    a, b = ctypes.c_void_p(0x10000), ctypes.c_void_p(0x20000)
    ok_args = lambda **kw: dict(dict(inp=a, ndim=2, shape=shp, fp=fp, st=None, fps=fps, org=None, op=0, mode=1, out=b), **kw)

    def grey(**kw):
        k = ok_args(**kw)
        return L.tm_grey_morph(k["inp"], k["ndim"], k["shape"], k["fp"], k["st"], k["fps"], k["org"], k["op"], k["mode"],
                               ctypes.c_float(0.0), k["out"], None)

    assert grey(inp=None) == E.ERR_INVALID_ARG and grey(out=None) == E.ERR_INVALID_ARG
    assert grey(op=2) == E.ERR_INVALID_ARG and grey(mode=5) == E.ERR_INVALID_ARG and grey(ndim=9) == E.ERR_INVALID_ARG
    assert grey(fp=(ctypes.c_uint8 * 9)()) == E.ERR_INVALID_ARG                      # no active position
    assert grey(org=(ctypes.c_int64 * 2)(2, 0)) == E.ERR_INVALID_ARG                 # centre outside the element
    assert grey(fps=(ctypes.c_int64 * 2)(0, 3)) == E.ERR_INVALID_ARG
    assert grey(out=ctypes.c_void_p(0x10010)) == E.ERR_INVALID_ARG                   # overlaps the input
    assert grey(shape=(ctypes.c_int64 * 4)(0, 1, 8, 8)) == E.OK                      # empty: nothing to do
    assert grey() == E.ERR_BAD_POINTER                                               # all fine but not device memory
    assert L.tm_binary_morph(a, 2, shp, fp, fps, None, 1, 0, b, None) == E.ERR_BAD_POINTER
    assert L.tm_binary_morph(a, 2, shp, fp, fps, None, 3, 0, b, None) == E.ERR_INVALID_ARG


def test_cdt_and_brute_force_argument_errors(L):
    E = binding
    shp = (ctypes.c_int64 * 4)(1, 1, 8, 8)
    a, b = ctypes.c_void_p(0x10000), ctypes.c_void_p(0x20000)
    assert L.tm_cdt(a, 2, shp, 0, b, None) == E.ERR_INVALID_ARG          # the Euclidean metric is tm_edt's
    assert L.tm_cdt(a, 2, shp, 3, b, None) == E.ERR_INVALID_ARG
    assert L.tm_cdt(None, 2, shp, 1, b, None) == E.ERR_INVALID_ARG
    assert L.tm_cdt(a, 2, shp, 1, ctypes.c_void_p(0x10020), None) == E.ERR_INVALID_ARG   # overlaps the mask
    assert L.tm_cdt(a, 2, (ctypes.c_int64 * 4)(1, 0, 8, 8), 1, b, None) == E.OK
    assert L.tm_cdt(a, 2, shp, 1, b, None) == E.ERR_BAD_POINTER
    assert L.tm_bfdt(a, 2, shp, None, 3, b, None) == E.ERR_INVALID_ARG
    assert L.tm_bfdt(a, 2, shp, (ctypes.c_double * 2)(1.0, -1.0), 0, b, None) == E.ERR_INVALID_ARG
    assert L.tm_bfdt(a, 5, (ctypes.c_int64 * 7)(1, 1, 2, 2, 2, 2, 2), None, 0, b, None) == E.ERR_UNSUPPORTED
    assert L.tm_bfdt(a, 2, (ctypes.c_int64 * 4)(1, 1, 8192, 4096), None, 0, b, None) == E.ERR_UNSUPPORTED  # > 2^24 voxels
    assert L.tm_bfdt(a, 2, shp, None, 2, b, None) == E.ERR_BAD_POINTER
