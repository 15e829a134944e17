"""CPU oracle for greyscale and binary erosion / dilation -- TEST INFRASTRUCTURE ONLY.

Plain numpy, written from the definition (paper, Section 2.1 "Covered transforms" and Section 2.3.1
"Fused morphology kernel"): the output at x combines the input at x + k - c over the active positions k of the
structuring element, c being its centre; values outside the image come from one of the five border rules of
scipy.ndimage (greyscale) or from a single border value (binary).  The image is padded once with the border
rule and the active positions are visited one by one: no blocking, no separable shortcuts.

  grey erosion    out(x) = min_k [ f(x + k - c) - s(k) ]
  grey dilation   out(x) = max_k [ f(x - k + c') + s(k) ]      (the reflected element, as SciPy defines it)
  binary erosion  out(x) = AND_k f(x + k - c),   binary dilation  out(x) = OR_k f(x - k + c')

with c = size // 2 + origin.  A dilation is written below as "reflect the element (origin negated, minus one on
even sizes, as SciPy does), then combine with max and + at the same kind of centre", so that the centre rule is
stated only once.  Arithmetic is float32 like the CUDA path (one subtraction or addition per tap; minima and
maxima are exact), so parity is bit-exact.

Pins (tests/test_morph_oracle_pins.py): scipy.ndimage.grey_erosion / grey_dilation / binary_erosion /
binary_dilation as black boxes over ranks 1..4, every border mode, even and odd element sizes, non-zero
origins; the duality dilation(f) = -erosion(-f) with the reflected element; flat 3^d elements against
scipy.ndimage.minimum_filter; monotonicity.  It shares no code with the CUDA library and never imports it.
"""
from __future__ import annotations

import numpy as np

MODES = ("constant", "reflect", "nearest", "mirror", "wrap")
_NP_PAD = {"reflect": "symmetric", "nearest": "edge", "mirror": "reflect", "wrap": "wrap"}


def _centres(fp_shape, origin):
    ndim = len(fp_shape)
    origin = (0,) * ndim if origin is None else tuple(int(o) for o in origin)
    return tuple(n // 2 + o for n, o in zip(fp_shape, origin))


def _pad(img, lo, hi, mode, cval):
    width = [(0, 0)] * (img.ndim - len(lo)) + list(zip(lo, hi))
    if mode == "constant":
        return np.pad(img, width, mode="constant", constant_values=cval)
    return np.pad(img, width, mode=_NP_PAD[mode])


def _combine(img, footprint, structure, centre, mode, cval, take_min):
    """out(x) = min or max over active k of img(x + k - centre) -/+ structure(k); img is (B, C, spatial...)."""
    footprint = np.asarray(footprint) != 0
    ndim = footprint.ndim
    spatial = img.shape[-ndim:]
    lo = [max(0, c) for c in centre]                                  # reach below 0
    hi = [max(0, n - 1 - c) for n, c in zip(footprint.shape, centre)]  # reach beyond the end
    pad = _pad(img, lo, hi, mode, cval)
    out = None
    for k in zip(*np.nonzero(footprint)):
        # x + k - centre, in padded coordinates: + lo
        sl = tuple(slice(l + kk - c, l + kk - c + n) for l, kk, c, n in zip(lo, k, centre, spatial))
        v = pad[(Ellipsis,) + sl]
        if structure is not None:
            s = np.float32(structure[k])
            v = (v - s) if take_min else (v + s)
        if out is None:
            out = v.copy()
        else:
            out = np.minimum(out, v) if take_min else np.maximum(out, v)
    if out is None:
        raise ValueError("the structuring element has no active position")
    return out


def _reflected(footprint, structure, origin):
    """The element reflected through its centre, with the origin SciPy uses for it (even sizes shift by one)."""
    footprint = np.asarray(footprint)
    ndim = footprint.ndim
    origin = [0] * ndim if origin is None else [int(o) for o in origin]
    flip = (slice(None, None, -1),) * ndim
    new_origin = [-o - (1 if n % 2 == 0 else 0) for o, n in zip(origin, footprint.shape)]
    return footprint[flip], (None if structure is None else np.asarray(structure)[flip]), new_origin


def grey_erosion(img, footprint, structure=None, mode="reflect", cval=0.0, origin=None):
    img = np.ascontiguousarray(img, dtype=np.float32)
    st = None if structure is None else np.asarray(structure, dtype=np.float32)
    return _combine(img, footprint, st, _centres(np.shape(footprint), origin), mode, np.float32(cval), True)


def grey_dilation(img, footprint, structure=None, mode="reflect", cval=0.0, origin=None):
    img = np.ascontiguousarray(img, dtype=np.float32)
    fp, st, org = _reflected(footprint, structure, origin)
    st = None if st is None else np.asarray(st, dtype=np.float32)
    return _combine(img, fp, st, _centres(fp.shape, org), mode, np.float32(cval), False)


def binary_erosion(img, structure, border_value=0, origin=None):
    img = (np.ascontiguousarray(img) != 0).astype(np.uint8)
    return _combine(img, structure, None, _centres(np.shape(structure), origin), "constant", np.uint8(1 if border_value else 0), True)


def binary_dilation(img, structure, border_value=0, origin=None):
    img = (np.ascontiguousarray(img) != 0).astype(np.uint8)
    fp, _, org = _reflected(structure, None, origin)
    return _combine(img, fp, None, _centres(fp.shape, org), "constant", np.uint8(1 if border_value else 0), False)
