"""Pins of the morphology oracle (oracle/morph_oracle.py) against scipy.ndimage as a black box and against
algebraic facts; none of these re-type the oracle's own formula."""
import numpy as np
import pytest

from oracle import morph_oracle as mo

ndi = pytest.importorskip("scipy.ndimage")

CASES = [
    ((17,), (3,), (0,)), ((17,), (4,), (0,)), ((17,), (5,), (1,)), ((9, 11), (3, 3), (0, 0)), ((9, 11), (2, 3), (0, 1)),
    ((9, 11), (4, 5), (-1, 1)), ((6, 7, 8), (3, 3, 3), (0, 0, 0)), ((6, 7, 8), (2, 3, 4), (0, -1, 1)),
    ((4, 5, 3, 6), (3, 2, 3, 3), (0, 0, 1, -1)), ((3, 4), (3, 3), (0, 0)),
]


def _inputs(shape, fp_shape, seed):
    rng = np.random.default_rng(seed)
    img = rng.normal(size=(2, 2) + shape).astype(np.float32)
    fp = rng.random(fp_shape) < 0.7
    fp.flat[rng.integers(0, fp.size)] = True
    st = rng.normal(size=fp_shape).astype(np.float32)
    return img, fp, st


@pytest.mark.parametrize("shape,fp_shape,origin", CASES)
@pytest.mark.parametrize("mode", mo.MODES)
@pytest.mark.parametrize("with_structure", [False, True])
def test_grey_operators_against_scipy(shape, fp_shape, origin, mode, with_structure):
    img, fp, st = _inputs(shape, fp_shape, 11 + len(shape))
    s = st if with_structure else None
    ero = mo.grey_erosion(img, fp, s, mode, 0.25, origin)
    dil = mo.grey_dilation(img, fp, s, mode, 0.25, origin)
    for b in range(2):
        for c in range(2):
            kw = dict(footprint=fp, structure=s, mode=mode, cval=0.25, origin=origin)
            np.testing.assert_array_equal(ero[b, c], ndi.grey_erosion(img[b, c], **kw))
            np.testing.assert_array_equal(dil[b, c], ndi.grey_dilation(img[b, c], **kw))


@pytest.mark.parametrize("shape,fp_shape,origin", CASES)
@pytest.mark.parametrize("border_value", [0, 1])
def test_binary_operators_against_scipy(shape, fp_shape, origin, border_value):
    rng = np.random.default_rng(5)
    img = (rng.random((2, 1) + shape) < 0.6).astype(np.uint8)
    _, fp, _ = _inputs(shape, fp_shape, 3)
    ero = mo.binary_erosion(img, fp, border_value, origin)
    dil = mo.binary_dilation(img, fp, border_value, origin)
    for b in range(2):
        np.testing.assert_array_equal(ero[b, 0].astype(bool), ndi.binary_erosion(img[b, 0], fp, border_value=border_value, origin=origin))
        np.testing.assert_array_equal(dil[b, 0].astype(bool), ndi.binary_dilation(img[b, 0], fp, border_value=border_value, origin=origin))


@pytest.mark.parametrize("mode", mo.MODES)
def test_duality_and_flat_filters(mode):
    img, fp, st = _inputs((7, 9, 8), (3, 3, 3), 2)
    flip = (slice(None, None, -1),) * 3
    # dilation by an element = - erosion of -f by the reflected element (odd sizes: same centre)
    np.testing.assert_array_equal(mo.grey_dilation(img, fp, st, mode, 0.0), -mo.grey_erosion(-img, fp[flip], st[flip], mode, 0.0))
    full = np.ones((3, 3, 3), dtype=bool)
    ero = mo.grey_erosion(img, full, None, mode, 0.5)
    for b in range(2):
        for c in range(2):
            np.testing.assert_array_equal(ero[b, c], ndi.minimum_filter(img[b, c], size=3, mode=mode, cval=0.5))
    # an element that contains its centre: erosion <= f <= dilation; a larger element erodes more
    fp[1, 1, 1] = True
    assert (mo.grey_erosion(img, fp, None, mode) <= img).all() and (mo.grey_dilation(img, fp, None, mode) >= img).all()
    assert (mo.grey_erosion(img, full, None, mode) <= mo.grey_erosion(img, fp, None, mode)).all()
