"""ctypes binding of the C-ABI library ``libtm_edt.so`` -- argument marshalling only.

Every step of the transform runs inside the CUDA library; PyTorch is used here for device memory and
streams.  There is no fallback: if the library cannot be loaded, or a call fails, an exception is
raised.  Entry points carry the names of the C functions declared in ``include/tm_edt.h``.
"""
from __future__ import annotations

import ctypes
import os
import threading
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtm_edt.so")
DEBUG_LIB_PATH = os.path.join(_HERE, "libtm_edt_debug.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_BAD_POINTER, ERR_ALLOC, ERR_CUDA, ERR_TOO_LARGE, ERR_DEBUG_CHECK = range(8)
MAX_DIMS = 8
MAX_EXTENT = 8192

EXPORTS = (
    "tm_edt", "tm_edt_ws", "tm_edt_ex", "tm_edt_ex_workspace_bytes", "tm_edt_host", "tm_edt_noalloc", "tm_edt_noalloc_max_scratch", "tm_edt_profile", "tm_edt_profile_ex", "tm_edt_workspace_bytes", "tm_edt_strerror",
    "tm_edt_last_cuda_error", "tm_edt_version", "tm_edt_last_launch_count", "tm_edt_trim_memory",
    "tm_edt_workspace_bytes_for", "tm_edt_reload_switches", "tm_edt_debug_build", "tm_edt_debug_last_violation",
    "tm_grey_morph", "tm_binary_morph", "tm_cdt", "tm_bfdt",
)

_lock = threading.Lock()
_lib = None


class TmEdtError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("tm_edt failed: %s (status %d)" % (message, status))
        self.status = status


def use_debug_library(on: bool = True) -> None:
    """Route every later call through the bounds-checked debug build (``buildlib.build(debug=True)``) or back."""
    global _lib, _use_debug
    with _lock:
        _use_debug = bool(on)
        _lib = None


_use_debug = False


def lib() -> ctypes.CDLL:
    """Open the CUDA library (once).  Raises if it has not been built: there is no other code path."""
    global _lib
    with _lock:
        if _lib is None:
            path = DEBUG_LIB_PATH if _use_debug else LIB_PATH
            if not os.path.exists(path):
                raise RuntimeError(
                    "CUDA library %s is missing; build it with `python -m paper_2608_24738_b200.buildlib`" % path
                )
            L = ctypes.CDLL(path)
            vp, i, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
            L.tm_edt.argtypes = [vp, i, vp, vp, vp, vp, vp, vp]
            L.tm_edt.restype = i
            L.tm_edt_ws.argtypes = [vp, i, vp, vp, vp, vp, vp, vp, sz, vp]
            L.tm_edt_ws.restype = i
            L.tm_edt_ex.argtypes = [vp, i, vp, vp, vp, vp, vp, vp, ctypes.c_uint, vp, sz, vp]
            L.tm_edt_ex.restype = i
            L.tm_edt_ex_workspace_bytes.argtypes = [i, vp, vp, ctypes.c_uint, i, i]
            L.tm_edt_ex_workspace_bytes.restype = sz
            L.tm_edt_host.argtypes = [vp, i, vp, vp, vp, vp, vp, vp]
            L.tm_edt_host.restype = i
            L.tm_edt_noalloc.argtypes = [vp, i, vp, vp, vp, vp, vp, vp]
            L.tm_edt_noalloc.restype = i
            L.tm_edt_noalloc_max_scratch.restype = sz
            L.tm_edt_profile.argtypes = [vp, i, vp, vp, vp, vp, vp, vp, sz, vp, i, vp, vp, vp, vp]
            L.tm_edt_profile.restype = i
            L.tm_edt_profile_ex.argtypes = [vp, i, vp, vp, vp, vp, vp, ctypes.c_uint, vp, sz, vp, i, vp, vp, vp, vp]
            L.tm_edt_profile_ex.restype = i
            L.tm_edt_workspace_bytes.argtypes = [i, vp]
            L.tm_edt_workspace_bytes.restype = sz
            L.tm_edt_workspace_bytes_for.argtypes = [i, vp, vp, i, i, i]
            L.tm_edt_workspace_bytes_for.restype = sz
            L.tm_edt_reload_switches.restype = None
            L.tm_edt_debug_build.restype = i
            L.tm_edt_debug_last_violation.argtypes = [vp, vp, vp]
            L.tm_edt_debug_last_violation.restype = ctypes.c_ulonglong
            L.tm_edt_strerror.argtypes = [i]
            L.tm_edt_strerror.restype = ctypes.c_char_p
            L.tm_edt_last_cuda_error.restype = i
            L.tm_edt_last_launch_count.restype = i
            L.tm_edt_version.restype = ctypes.c_char_p
            L.tm_edt_trim_memory.restype = i
            L.tm_grey_morph.argtypes = [vp, i, vp, vp, vp, vp, vp, i, i, ctypes.c_float, vp, vp]
            L.tm_grey_morph.restype = i
            L.tm_binary_morph.argtypes = [vp, i, vp, vp, vp, vp, i, i, vp, vp]
            L.tm_binary_morph.restype = i
            L.tm_cdt.argtypes = [vp, i, vp, i, vp, vp]
            L.tm_cdt.restype = i
            L.tm_bfdt.argtypes = [vp, i, vp, vp, i, vp, vp]
            L.tm_bfdt.restype = i
            _lib = L
    return _lib


def tm_edt_strerror(status: int) -> str:
    return lib().tm_edt_strerror(int(status)).decode()


def tm_edt_version() -> str:
    return lib().tm_edt_version().decode()


def tm_edt_last_cuda_error() -> int:
    return int(lib().tm_edt_last_cuda_error())


def tm_edt_trim_memory() -> None:
    """Give the library's pooled scratch memory of the current device back to the driver."""
    _check(int(lib().tm_edt_trim_memory()))


def tm_edt_last_launch_count() -> int:
    return int(lib().tm_edt_last_launch_count())


def _shape_array(shape: Sequence[int]):
    return (ctypes.c_int64 * len(shape))(*[int(s) for s in shape])


def _sampling_array(sampling, ndim):
    if sampling is None:
        return None
    vals = [float(s) for s in sampling]
    if len(vals) != ndim:
        raise ValueError("sampling needs one entry per spatial axis")
    return (ctypes.c_double * ndim)(*vals)


def tm_edt_workspace_bytes(shape: Sequence[int]) -> int:
    """shape = (B, C, n_0 .. n_{d-1})."""
    n = int(lib().tm_edt_workspace_bytes(len(shape) - 2, _shape_array(shape)))
    if n == ctypes.c_size_t(-1).value:
        raise TmEdtError(ERR_INVALID_ARG, "invalid or unsupported shape")
    return n


def tm_edt_workspace_bytes_for(shape: Sequence[int], sampling=None, want_dist=True, want_sqdist=False,
                               want_indices=False) -> int:
    """Scratch bytes of one particular call: shape = (B, C, n_0 .. n_{d-1}), its sampling and requested outputs."""
    ndim = len(shape) - 2
    n = int(lib().tm_edt_workspace_bytes_for(ndim, _shape_array(shape), _sampling_array(sampling, ndim), int(want_dist),
                                             int(want_sqdist), int(want_indices)))
    if n == ctypes.c_size_t(-1).value:
        raise TmEdtError(ERR_INVALID_ARG, "invalid or unsupported shape")
    return n


def tm_edt_debug_build() -> bool:
    return bool(lib().tm_edt_debug_build())


def tm_edt_debug_last_violation():
    """(count, site code, index, bound) of the bounds violations the calling thread's last call recorded."""
    c, i, l = ctypes.c_longlong(0), ctypes.c_longlong(0), ctypes.c_longlong(0)
    n = int(lib().tm_edt_debug_last_violation(ctypes.byref(c), ctypes.byref(i), ctypes.byref(l)))
    return n, int(c.value), int(i.value), int(l.value)


def tm_edt_reload_switches() -> None:
    """Read the library's debug switches from the environment again (they are otherwise read once)."""
    lib().tm_edt_reload_switches()


def _raw_stream(stream) -> Optional[int]:
    import torch

    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _check(status: int) -> None:
    if status != OK:
        raise TmEdtError(status, tm_edt_strerror(status))


FLAG_VIRTUAL_BACKGROUND = 1
FLAG_FLAT_INDEX = 2
FLAG_DIST_F64 = 4


def _contiguous_on(t, stream):
    """A contiguous copy of a CUDA tensor for kernels that will run on ``stream``.

    The copy is made on that stream (after what the current stream has queued, which may still be producing ``t``),
    so it is complete before the kernels read it and its memory is not handed out again before they have run."""
    import torch

    if t.is_contiguous():
        return t
    if not t.is_cuda or stream is None:
        return t.contiguous()
    cur = torch.cuda.current_stream(t.device)
    if stream == cur:
        return t.contiguous()
    stream.wait_stream(cur)
    with torch.cuda.stream(stream):
        return t.contiguous()


def _prepare(mask, sampling, return_distances, return_sqdist, return_indices, distances, sqdist, indices, device,
             flat_index=False, dist_f64=False, keep_strides=False, stream=None):
    import torch

    if mask.dim() < 3:
        raise ValueError("mask must be shaped (B, C, spatial...)")
    if mask.dtype == torch.bool:
        mask = mask.view(torch.uint8)
    if mask.dtype != torch.uint8:
        raise TypeError("mask must be uint8 or bool")
    if not mask.is_contiguous() and not keep_strides:
        mask = _contiguous_on(mask, stream)
    shape = tuple(mask.shape)
    ndim = len(shape) - 2

    def out(buf, want, dtype, shp):
        if buf is not None:
            if buf.dtype != dtype or tuple(buf.shape) != tuple(shp) or not buf.is_contiguous():
                raise ValueError("pre-allocated output has the wrong dtype, shape or layout")
            return buf
        return torch.empty(shp, dtype=dtype, device=device, pin_memory=(device == "cpu_pinned")) if want else None

    dev = mask.device if device is None else device
    if dev == "cpu_pinned":
        mk = lambda want, dtype, shp, buf: buf if buf is not None else (
            torch.empty(shp, dtype=dtype, pin_memory=True) if want else None)
    else:
        mk = lambda want, dtype, shp, buf: out(buf, want, dtype, shp)
    d = mk(return_distances, torch.float64 if dist_f64 else torch.float32, shape, distances)
    s = mk(return_sqdist, torch.int64, shape, sqdist)
    x = mk(return_indices, torch.int64, shape if flat_index else shape[:2] + (ndim,) + shape[2:], indices)
    return mask, shape, ndim, d, s, x


def _p(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def tm_edt_ex_workspace_bytes(shape, strides=None, flags=0, with_distances=True, with_indices=False) -> int:
    """Scratch bytes of a ``tm_edt_ex`` call; ``strides`` are BYTE strides of the (B, C, spatial...) mask or None."""
    L = lib()
    st = None if strides is None else (ctypes.c_int64 * len(strides))(*[int(v) for v in strides])
    n = L.tm_edt_ex_workspace_bytes(len(shape) - 2, _shape_array(shape), st, ctypes.c_uint(flags), int(with_distances),
                                    int(with_indices))
    if n == ctypes.c_size_t(-1).value:
        raise TmEdtError(ERR_INVALID_ARG, "invalid or unsupported shape / strides")
    return int(n)


def tm_edt(mask, sampling=None, return_distances=True, return_indices=False, return_sqdist=False,
           distances=None, indices=None, sqdist=None, workspace=None, stream=None,
           virtual_background=False, flat_index=False, dist_f64=False, keep_strides=False):
    """Distance transform of a CUDA mask tensor (B, C, spatial...), uint8 or bool.

    Returns a dict with the requested tensors among ``dist`` (float32), ``sq`` (int64, unit sampling
    only) and ``idx`` (int64, (B, C, ndim, spatial...)).  With ``workspace`` (a CUDA uint8 tensor of at
    least ``tm_edt_workspace_bytes(mask.shape)`` bytes) the call goes through ``tm_edt_ws`` and allocates
    nothing; otherwise through ``tm_edt``.  Work is enqueued on ``stream`` (default: current stream).
    The remaining keywords select the variants of ``tm_edt_ex``: ``virtual_background`` (SciPy's values for images
    without background), ``flat_index`` (``idx`` as one linear index per voxel, shaped like the mask), ``dist_f64``
    (``dist`` as float64) and ``keep_strides`` (a non-contiguous mask is passed with its strides and gathered by
    the library instead of being made contiguous here).
    """
    L = lib()
    if not mask.is_cuda:
        raise ValueError("mask must be a CUDA tensor (use tm_edt_host for host buffers)")
    mask, shape, ndim, d, s, x = _prepare(
        mask, sampling, return_distances, return_sqdist, return_indices, distances, sqdist, indices, mask.device,
        flat_index=flat_index, dist_f64=dist_f64, keep_strides=keep_strides, stream=stream)
    shp, smp, st = _shape_array(shape), _sampling_array(sampling, ndim), _raw_stream(stream)
    flags = ((FLAG_VIRTUAL_BACKGROUND if virtual_background else 0) | (FLAG_FLAT_INDEX if flat_index else 0)
             | (FLAG_DIST_F64 if dist_f64 else 0))
    strided = keep_strides and not mask.is_contiguous()
    if flags or strided:
        nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        strides = (ctypes.c_int64 * len(shape))(*[int(v) for v in mask.stride()]) if strided else None
        rc = L.tm_edt_ex(_p(mask), ndim, shp, strides, smp, _p(d), _p(s), _p(x), ctypes.c_uint(flags), _p(workspace),
                         ctypes.c_size_t(nbytes), st)
    elif workspace is None:
        rc = L.tm_edt(_p(mask), ndim, shp, smp, _p(d), _p(s), _p(x), st)
    else:
        rc = L.tm_edt_ws(_p(mask), ndim, shp, smp, _p(d), _p(s), _p(x), _p(workspace),
                         ctypes.c_size_t(workspace.numel() * workspace.element_size()), st)
    _check(rc)
    return {"dist": d, "sq": s, "idx": x}


def tm_edt_noalloc_max_scratch() -> int:
    return int(lib().tm_edt_noalloc_max_scratch())


def tm_edt_noalloc(mask, sampling=None, return_distances=True, return_indices=False, return_sqdist=False,
                   distances=None, indices=None, sqdist=None, stream=None):
    """The transform through the entry point that never allocates device memory: scratch comes from a
    fixed array inside the library, for hosts that may not call cudaMalloc once they are running (fixed
    memory budgets, foreign allocators).  Pass pre-allocated ``distances`` / ``sqdist`` / ``indices`` if
    the outputs, too, must not be allocated here.  Problems needing more scratch than
    ``tm_edt_noalloc_max_scratch()`` raise ``TmEdtError`` with status ``ERR_TOO_LARGE``.  Calls that overlap
    on the GPU share the array and would race; keep them ordered on one stream."""
    L = lib()
    if not mask.is_cuda:
        raise ValueError("mask must be a CUDA tensor")
    mask, shape, ndim, d, s, x = _prepare(
        mask, sampling, return_distances, return_sqdist, return_indices, distances, sqdist, indices, mask.device, stream=stream)
    rc = L.tm_edt_noalloc(_p(mask), ndim, _shape_array(shape), _sampling_array(sampling, ndim), _p(d), _p(s), _p(x),
                          _raw_stream(stream))
    _check(rc)
    return {"dist": d, "sq": s, "idx": x}


def tm_edt_host(mask, sampling=None, return_distances=True, return_indices=False, return_sqdist=False,
                distances=None, indices=None, sqdist=None, stream=None):
    """Same transform for HOST tensors (pinned for asynchronous copies): the C library copies the mask to
    the device, runs, and copies the outputs back, all on ``stream``; the caller synchronises."""
    L = lib()
    if mask.is_cuda:
        raise ValueError("tm_edt_host takes host tensors")
    mask, shape, ndim, d, s, x = _prepare(
        mask, sampling, return_distances, return_sqdist, return_indices, distances, sqdist, indices, "cpu_pinned", stream=stream)
    rc = L.tm_edt_host(_p(mask), ndim, _shape_array(shape), _sampling_array(sampling, ndim), _p(d), _p(s), _p(x),
                       _raw_stream(stream))
    _check(rc)
    return {"dist": d, "sq": s, "idx": x}


def tm_edt_profile(mask, sampling=None, return_distances=True, return_indices=False, return_sqdist=False,
                   distances=None, indices=None, sqdist=None, workspace=None, stream=None, flags=0):
    """tm_edt_ws with per-kernel device times: returns (outputs dict, [(kernel label, milliseconds, bytes the launch must move), ...]).
    Blocks until the work is done.  ``workspace`` is required when the shape needs scratch."""
    import torch

    L = lib()
    mask, shape, ndim, d, s, x = _prepare(
        mask, sampling, return_distances, return_sqdist, return_indices, distances, sqdist, indices, mask.device,
        flat_index=bool(flags & FLAG_FLAT_INDEX), stream=stream)
    if workspace is None:
        workspace = torch.empty(max(1, tm_edt_workspace_bytes(shape)), dtype=torch.uint8, device=mask.device)
    kmax = 32
    ms = (ctypes.c_float * kmax)()
    nbytes = (ctypes.c_double * kmax)()
    names = ctypes.create_string_buffer(48 * kmax)
    n = ctypes.c_int(0)
    rc = L.tm_edt_profile_ex(_p(mask), ndim, _shape_array(shape), _sampling_array(sampling, ndim), _p(d), _p(s), _p(x),
                             ctypes.c_uint(flags), _p(workspace), ctypes.c_size_t(workspace.numel()), _raw_stream(stream),
                             kmax, ms, nbytes, names, ctypes.byref(n))
    _check(rc)
    out = [(names.raw[48 * k: 48 * k + 48].split(b"\0", 1)[0].decode(), float(ms[k]), float(nbytes[k]))
           for k in range(n.value)]
    return {"dist": d, "sq": s, "idx": x}, out


class PreparedCall:
    """A tm_edt_ws call with its arguments marshalled once, for callers that repeat it (benchmarks, loops)."""

    def __init__(self, mask, sampling=None, distances=None, sqdist=None, indices=None, workspace=None, flags=0):
        import torch

        self._L = lib()
        self.flags = int(flags)
        self.mask, self.shape, self.ndim, self.d, self.s, self.x = _prepare(
            mask, sampling, distances is not None, sqdist is not None, indices is not None, distances, sqdist,
            indices, mask.device, flat_index=bool(self.flags & FLAG_FLAT_INDEX))
        need = tm_edt_workspace_bytes(self.shape)
        if workspace is None:
            workspace = torch.empty(max(1, need), dtype=torch.uint8, device=mask.device)
        self.ws = workspace
        shp, smp = _shape_array(self.shape), _sampling_array(sampling, self.ndim)
        outs = (_p(self.d), _p(self.s), _p(self.x))
        tail = (_p(self.ws), ctypes.c_size_t(self.ws.numel()))
        if self.flags:
            self._fn = self._L.tm_edt_ex
            self._args = (_p(self.mask), self.ndim, shp, None, smp) + outs + (ctypes.c_uint(self.flags),) + tail
        else:
            self._fn = self._L.tm_edt_ws
            self._args = (_p(self.mask), self.ndim, shp, smp) + outs + tail

    def __call__(self, stream_ptr):
        rc = self._fn(*self._args, stream_ptr)
        if rc != OK:
            _check(rc)


MORPH_MODES = {"constant": 0, "reflect": 1, "nearest": 2, "mirror": 3, "wrap": 4}


class PreparedMorph:
    """A tm_grey_morph / tm_binary_morph call with its arguments marshalled once, for callers that repeat it."""

    def __init__(self, image, footprint, structure=None, op="erosion", mode="reflect", cval=0.0, origin=None, out=None,
                 border_value=0):
        import numpy as np
        import torch

        L = lib()
        binary = image.dtype in (torch.uint8, torch.bool)
        if image.dtype == torch.bool:
            image = image.view(torch.uint8)
        if not image.is_cuda or image.dim() < 3 or not image.is_contiguous():
            raise ValueError("image must be a contiguous CUDA tensor shaped (B, C, spatial...)")
        ndim = image.dim() - 2
        fp, fps = _element(footprint, ndim)
        st = None if structure is None else np.ascontiguousarray(structure, dtype=np.float32)
        self.image, self.out = image, (torch.empty_like(image) if out is None else out)
        self._keep = (fp, fps, st, _shape_array(tuple(image.shape)), _origin(origin, ndim))
        opc = {"erosion": 0, "dilation": 1}[op]
        if binary:
            self._fn = L.tm_binary_morph
            self._args = (_p(image), ndim, self._keep[3], fp.ctypes.data_as(ctypes.c_void_p), fps, self._keep[4], opc,
                          int(bool(border_value)), _p(self.out))
        else:
            self._fn = L.tm_grey_morph
            self._args = (_p(image), ndim, self._keep[3], fp.ctypes.data_as(ctypes.c_void_p),
                          None if st is None else st.ctypes.data_as(ctypes.c_void_p), fps, self._keep[4], opc,
                          MORPH_MODES[mode], ctypes.c_float(cval), _p(self.out))

    def __call__(self, stream_ptr):
        rc = self._fn(*self._args, stream_ptr)
        if rc != OK:
            _check(rc)


def _element(footprint, ndim):
    import numpy as np

    fp = np.ascontiguousarray(np.asarray(footprint) != 0, dtype=np.uint8)
    if fp.ndim != ndim:
        raise ValueError("the structuring element needs one axis per spatial axis")
    return fp, (ctypes.c_int64 * ndim)(*fp.shape)


def _origin(origin, ndim):
    return None if origin is None else (ctypes.c_int64 * ndim)(*[int(o) for o in origin])


def tm_grey_morph(image, footprint, structure=None, op="erosion", mode="reflect", cval=0.0, origin=None, out=None,
                  stream=None):
    """Greyscale erosion or dilation of a CUDA float32 tensor (B, C, spatial...) with scipy.ndimage conventions:
    ``footprint`` (array-like, one axis per spatial axis) marks the active positions, ``structure`` (same shape,
    optional) is the additive structuring function, ``mode`` one of constant / reflect / nearest / mirror / wrap."""
    import numpy as np
    import torch

    L = lib()
    if not image.is_cuda or image.dtype != torch.float32 or image.dim() < 3:
        raise ValueError("image must be a CUDA float32 tensor shaped (B, C, spatial...)")
    image = _contiguous_on(image, stream)
    ndim = image.dim() - 2
    fp, fps = _element(footprint, ndim)
    st = None
    if structure is not None:
        st = np.ascontiguousarray(structure, dtype=np.float32)
        if st.shape != fp.shape:
            raise ValueError("structure and footprint differ in shape")
    if out is None:
        out = torch.empty_like(image)
    rc = L.tm_grey_morph(_p(image), ndim, _shape_array(tuple(image.shape)), fp.ctypes.data_as(ctypes.c_void_p),
                         None if st is None else st.ctypes.data_as(ctypes.c_void_p), fps, _origin(origin, ndim),
                         {"erosion": 0, "dilation": 1}[op], MORPH_MODES[mode], ctypes.c_float(cval), _p(out),
                         _raw_stream(stream))
    _check(rc)
    return out


def tm_binary_morph(mask, structure, op="erosion", border_value=0, origin=None, out=None, stream=None):
    """Binary erosion or dilation of a CUDA uint8 / bool tensor (B, C, spatial...); returns uint8 holding 0 or 1."""
    import torch

    L = lib()
    if not mask.is_cuda or mask.dim() < 3:
        raise ValueError("mask must be a CUDA tensor shaped (B, C, spatial...)")
    if mask.dtype == torch.bool:
        mask = mask.view(torch.uint8)
    if mask.dtype != torch.uint8:
        raise TypeError("mask must be uint8 or bool")
    mask = _contiguous_on(mask, stream)
    ndim = mask.dim() - 2
    fp, fps = _element(structure, ndim)
    if out is None:
        out = torch.empty_like(mask)
    rc = L.tm_binary_morph(_p(mask), ndim, _shape_array(tuple(mask.shape)), fp.ctypes.data_as(ctypes.c_void_p), fps,
                           _origin(origin, ndim), {"erosion": 0, "dilation": 1}[op], int(bool(border_value)), _p(out),
                           _raw_stream(stream))
    _check(rc)
    return out


METRICS = {"euclidean": 0, "taxicab": 1, "chessboard": 2}


def _mask_u8(mask, stream=None):
    import torch

    if not mask.is_cuda or mask.dim() < 3:
        raise ValueError("mask must be a CUDA tensor shaped (B, C, spatial...)")
    if mask.dtype == torch.bool:
        mask = mask.view(torch.uint8)
    if mask.dtype != torch.uint8:
        raise TypeError("mask must be uint8 or bool")
    return _contiguous_on(mask, stream)


def tm_cdt(mask, metric="chessboard", out=None, stream=None):
    """Taxicab or chessboard distance transform (int32, -1 for an image without background), the values of
    scipy.ndimage.distance_transform_cdt."""
    import torch

    L = lib()
    mask = _mask_u8(mask, stream)
    if out is None:
        out = torch.empty(mask.shape, dtype=torch.int32, device=mask.device)
    _check(L.tm_cdt(_p(mask), mask.dim() - 2, _shape_array(tuple(mask.shape)), METRICS[metric], _p(out), _raw_stream(stream)))
    return out


def tm_bfdt(mask, sampling=None, metric="euclidean", out=None, stream=None):
    """Brute-force distance transform (float32): every voxel against every background voxel; ranks 1..4."""
    import torch

    L = lib()
    mask = _mask_u8(mask, stream)
    ndim = mask.dim() - 2
    if out is None:
        out = torch.empty(mask.shape, dtype=torch.float32, device=mask.device)
    _check(L.tm_bfdt(_p(mask), ndim, _shape_array(tuple(mask.shape)), _sampling_array(sampling, ndim), METRICS[metric],
                     _p(out), _raw_stream(stream)))
    return out
