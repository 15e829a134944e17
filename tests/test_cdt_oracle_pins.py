"""Pins of the taxicab / chessboard oracle against scipy.ndimage.distance_transform_cdt, its own brute-force form,
closed forms and the metric ordering."""
import numpy as np
import pytest

import oracle
from oracle import cdt_oracle as co

ndi = pytest.importorskip("scipy.ndimage")
SHAPES = [(9,), (7, 8), (5, 6, 7), (3, 4, 3, 5), (2, 3, 2, 3, 2, 3)]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("metric", ["taxicab", "chessboard"])
@pytest.mark.parametrize("p_fg", [0.5, 0.95])
def test_forms_agree_and_match_scipy(shape, metric, p_fg):
    rng = np.random.default_rng(len(shape) * 7 + int(p_fg * 10))
    mask = (rng.random((2, 2) + shape) < p_fg).astype(np.uint8)
    mask[1, 1] = 1  # an image without background
    sep = co.separable(mask, metric)
    assert sep.dtype == np.int32 and (sep[1, 1] == -1).all()
    assert np.array_equal(sep, co.brute(mask, metric))
    for b in range(2):
        for c in range(2):
            assert np.array_equal(sep[b, c], ndi.distance_transform_cdt(mask[b, c], metric=metric))


@pytest.mark.parametrize("ndim", [1, 2, 3, 4])
def test_single_background_voxel_and_metric_ordering(ndim):
    shape = (7, 6, 5, 4)[:ndim]
    site = tuple(n // 3 for n in shape)
    mask = np.ones((1, 1) + shape, dtype=np.uint8)
    mask[(0, 0) + site] = 0
    grid = np.meshgrid(*[np.arange(n) for n in shape], indexing="ij")
    diff = [np.abs(g - s) for g, s in zip(grid, site)]
    assert np.array_equal(co.separable(mask, "taxicab")[0, 0], sum(diff))
    assert np.array_equal(co.separable(mask, "chessboard")[0, 0], np.maximum.reduce(diff))
    rng = np.random.default_rng(ndim)
    m = (rng.random((1, 1) + shape) < 0.8).astype(np.uint8)
    m[(0, 0) + site] = 0
    d1, dinf = co.separable(m, "taxicab").astype(np.float64), co.separable(m, "chessboard").astype(np.float64)
    d2 = oracle.sep(m, None, want_idx=False)["dist"]
    assert (dinf <= d2 + 1e-12).all() and (d2 <= d1 + 1e-12).all() and (d1 <= ndim * dinf).all()


def test_weighted_brute_force():
    """Anisotropic taxicab / chessboard distances (brute force only): one background voxel, closed form."""
    mask = np.ones((1, 1, 5, 6), dtype=np.uint8)
    mask[0, 0, 1, 4] = 0
    yy, xx = np.meshgrid(np.arange(5), np.arange(6), indexing="ij")
    np.testing.assert_allclose(co.brute(mask, "taxicab", (2.5, 0.5))[0, 0], 2.5 * np.abs(yy - 1) + 0.5 * np.abs(xx - 4))
    np.testing.assert_allclose(co.brute(mask, "chessboard", (2.5, 0.5))[0, 0], np.maximum(2.5 * np.abs(yy - 1), 0.5 * np.abs(xx - 4)))
    assert np.isinf(co.brute(np.ones((1, 1, 3, 3), np.uint8), "taxicab", (1.0, 2.0))).all()
