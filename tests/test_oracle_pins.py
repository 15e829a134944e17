"""Pins for the CPU oracle (no GPU): hand-computed fixtures, closed forms, brute force on small
inputs, invariants and SciPy as a black box.  Each is chosen so that a dropped term, a wrong sign or
index, or a swapped axis in the oracle fails at least one of them."""
import itertools
import os
import zlib

import numpy as np
import pytest

import oracle
from tests import checker
from tests.conftest import GOLDEN_DIR, read_golden

GOLDEN = read_golden(os.path.join(GOLDEN_DIR, "edt_hand_cases.txt"))


def _unit(s):
    return s is None or all(float(v) == 1.0 for v in s)


@pytest.mark.parametrize("case", GOLDEN, ids=[c["name"] for c in GOLDEN])
@pytest.mark.parametrize("routine", ["brute", "sep"])
def test_hand_computed_fixtures(case, routine):
    fn = getattr(oracle, routine)
    r = fn(case["mask"], case["sampling"])
    assert np.array_equal(np.isinf(r["sqf"]), np.isinf(case["sq"]))
    fin = np.isfinite(case["sq"])
    np.testing.assert_allclose(r["sqf"][fin], case["sq"][fin], rtol=1e-14, atol=0)
    np.testing.assert_allclose(r["dist"][fin], np.sqrt(case["sq"][fin]), rtol=1e-14)
    if _unit(case["sampling"]):
        exp = np.where(fin, case["sq"], 0).astype(np.int64)
        exp[~fin] = np.iinfo(np.int64).max
        assert np.array_equal(r["sq"], exp)
    if not fin.all():
        assert (r["idx"] == -1).all()
        assert np.isinf(r["dist"]).all()


SHAPES = [
    (1, 1, 17), (2, 1, 1), (1, 2, 7, 5), (1, 1, 1, 9), (1, 1, 9, 1), (2, 2, 5, 4, 3), (1, 1, 3, 1, 4),
    (1, 1, 3, 4, 2, 3), (1, 1, 2, 3, 2, 3, 2), (1, 1, 2, 2, 3, 2, 2, 3), (1, 1, 2, 2, 2, 2, 3, 2, 2),
    (1, 1, 2, 2, 2, 2, 2, 2, 2, 3), (1, 1, 13, 11), (1, 1, 2, 31),
]


def _sampling_for(ndim, kind):
    if kind == "unit":
        return None
    return tuple(0.5 + 0.37 * ((3 * k + 1) % 5) for k in range(ndim))


@pytest.mark.parametrize("shape", SHAPES, ids=["x".join(map(str, s)) for s in SHAPES])
@pytest.mark.parametrize("p_fg", [0.05, 0.5, 0.95])
@pytest.mark.parametrize("kind", ["unit", "sampled"])
def test_sep_equals_brute_force(shape, p_fg, kind):
    rng = np.random.default_rng(zlib.crc32(repr((shape, int(p_fg * 100), kind)).encode()))
    mask = (rng.random(shape) < p_fg).astype(np.uint8)
    sampling = _sampling_for(len(shape) - 2, kind)
    b = oracle.brute(mask, sampling)
    s = oracle.sep(mask, sampling)
    assert np.array_equal(np.isinf(b["sqf"]), np.isinf(s["sqf"]))
    fin = np.isfinite(b["sqf"])
    if kind == "unit":
        assert np.array_equal(b["sq"], s["sq"])
        assert np.array_equal(b["dist"], s["dist"])
    else:
        np.testing.assert_allclose(s["sqf"][fin], b["sqf"][fin], rtol=1e-13)
    for r in (b, s):
        checker.check_indices(r["idx"], mask, b, sampling, tol=1e-12)
    # zero exactly on the background, at least the smallest step elsewhere
    assert ((b["sqf"] == 0) == (mask == 0)).all() or mask.all(axis=tuple(range(2, mask.ndim))).any()
    wmin = 1.0 if sampling is None else min(sampling)
    fg = (mask != 0) & fin
    assert (s["dist"][fg] >= wmin - 1e-12).all()
    assert (s["dist"][mask == 0] == 0).all()


def test_config1_every_voxel_against_brute_force():
    from paper_2608_24738_b200 import workloads

    w = workloads.config1()
    b = oracle.brute(w.mask, w.sampling)
    s = oracle.sep(w.mask, w.sampling)
    assert np.array_equal(b["sq"], s["sq"])
    checker.check_indices(s["idx"], w.mask, b, None)


@pytest.mark.parametrize("ndim", [1, 2, 3, 4, 5, 8])
@pytest.mark.parametrize("routine", ["brute", "sep"])
def test_single_background_voxel_closed_form(ndim, routine):
    """One background voxel z: dist(x) = sqrt(sum (w_k (x_k - z_k))^2) and every index is z."""
    spatial = tuple([5, 4, 3, 3, 2, 2, 2, 2][:ndim])
    rng = np.random.default_rng(100 + ndim)
    z = tuple(int(rng.integers(0, n)) for n in spatial)
    sampling = tuple(0.7 + 0.45 * k for k in range(ndim))
    mask = np.ones((1, 1) + spatial, dtype=np.uint8)
    mask[(0, 0) + z] = 0
    r = getattr(oracle, routine)(mask, sampling)
    grid = checker.coords_grid(spatial)
    expect = np.zeros(spatial)
    for k in range(ndim):
        expect = expect + (sampling[k] * (grid[k] - z[k])) ** 2
    np.testing.assert_allclose(r["sqf"][0, 0], expect, rtol=1e-13)
    np.testing.assert_allclose(r["dist"][0, 0], np.sqrt(expect), rtol=1e-13)
    for k in range(ndim):
        assert (r["idx"][0, 0, k] == z[k]).all()
    # same mask, unit sampling: exact integers
    r1 = getattr(oracle, routine)(mask, None)
    e1 = np.zeros(spatial, dtype=np.int64)
    for k in range(ndim):
        e1 = e1 + (grid[k] - z[k]) ** 2
    assert np.array_equal(r1["sq"][0, 0], e1)


@pytest.mark.parametrize("axis", [0, 1, 2])
@pytest.mark.parametrize("routine", ["brute", "sep"])
def test_half_space_closed_form(axis, routine):
    """Background = {x_a < t}: dist = w_a (x_a - t + 1), idx_a = t - 1, other components the voxel's own."""
    spatial, t = (6, 5, 7), 2
    sampling = (1.3, 0.6, 2.0)
    mask = np.ones((1, 1) + spatial, dtype=np.uint8)
    sl = [slice(None)] * 5
    sl[2 + axis] = slice(0, t)
    mask[tuple(sl)] = 0
    r = getattr(oracle, routine)(mask, sampling)
    grid = checker.coords_grid(spatial)
    xa = np.broadcast_to(grid[axis], spatial)
    expect = np.where(xa < t, 0.0, sampling[axis] * (xa - t + 1))
    np.testing.assert_allclose(r["dist"][0, 0], expect, rtol=1e-13)
    for k in range(3):
        own = np.broadcast_to(grid[k], spatial)
        if k == axis:
            assert np.array_equal(r["idx"][0, 0, k], np.where(xa < t, xa, t - 1))
        else:
            assert np.array_equal(r["idx"][0, 0, k], own)


@pytest.mark.parametrize("kind", ["unit", "sampled"])
def test_axis_permutation_and_flip(kind):
    """Permuting / flipping the axes of the mask together with the sampling permutes / flips the result."""
    rng = np.random.default_rng(7)
    spatial = (5, 6, 4)
    mask = (rng.random((2, 1) + spatial) < 0.8).astype(np.uint8)
    sampling = None if kind == "unit" else (1.7, 0.6, 1.1)
    base = oracle.sep(mask, sampling, want_idx=False)
    for perm in itertools.permutations(range(3)):
        pm = np.ascontiguousarray(mask.transpose((0, 1) + tuple(2 + p for p in perm)))
        ps = None if sampling is None else tuple(sampling[p] for p in perm)
        r = oracle.sep(pm, ps, want_idx=False)
        exp = base["sqf"].transpose((0, 1) + tuple(2 + p for p in perm))
        if kind == "unit":
            assert np.array_equal(r["sq"], base["sq"].transpose((0, 1) + tuple(2 + p for p in perm)))
        else:
            np.testing.assert_allclose(r["sqf"], exp, rtol=1e-13)
    for ax in range(3):
        fm = np.ascontiguousarray(np.flip(mask, axis=2 + ax))
        r = oracle.sep(fm, sampling, want_idx=False)
        if kind == "unit":
            assert np.array_equal(r["sq"], np.flip(base["sq"], axis=2 + ax))
        else:
            np.testing.assert_allclose(r["sqf"], np.flip(base["sqf"], axis=2 + ax), rtol=1e-13)


def test_axis_order_of_nested_minima_is_free():
    rng = np.random.default_rng(11)
    mask = (rng.random((1, 2, 6, 5, 7)) < 0.85).astype(np.uint8)
    ref = oracle.sep(mask, None)
    for order in itertools.permutations(range(3)):
        r = oracle.sep_axes(mask, order, None)
        assert np.array_equal(r["sq"], ref["sq"])
    samp = (2.5, 0.8, 1.0)
    ref = oracle.sep(mask, samp)
    for order in itertools.permutations(range(3)):
        r = oracle.sep_axes(mask, order, samp)
        np.testing.assert_allclose(r["sqf"], ref["sqf"], rtol=1e-13)


def test_partial_axes_is_lower_dimensional_transform():
    """Nested minima over the last axis only = the 1-D transform of every line."""
    rng = np.random.default_rng(13)
    mask = (rng.random((1, 1, 4, 9)) < 0.7).astype(np.uint8)
    part = oracle.sep_axes(mask, [1], (3.0, 0.5))
    lines = oracle.sep(mask.reshape(4, 1, 9), (0.5,))
    assert np.array_equal(np.isinf(part["sqf"]).reshape(4, 1, 9), np.isinf(lines["sqf"]))
    fin = np.isfinite(lines["sqf"])
    np.testing.assert_allclose(part["sqf"].reshape(4, 1, 9)[fin], lines["sqf"][fin], rtol=1e-14)


def test_neighbour_differences_bounded_by_step():
    rng = np.random.default_rng(17)
    mask = (rng.random((1, 1, 12, 9, 10)) < 0.9).astype(np.uint8)
    samp = (2.5, 0.8, 1.0)
    d = oracle.sep(mask, samp, want_idx=False)["dist"][0, 0]
    for k in range(3):
        assert (np.abs(np.diff(d, axis=k)) <= samp[k] + 1e-12).all()


def test_more_background_never_increases_distance():
    rng = np.random.default_rng(19)
    mask = (rng.random((1, 1, 10, 11, 6)) < 0.9).astype(np.uint8)
    more = mask.copy()
    more[rng.random(mask.shape) < 0.05] = 0
    a = oracle.sep(mask, (1.0, 1.5, 0.5), want_idx=False)["sqf"]
    b = oracle.sep(more, (1.0, 1.5, 0.5), want_idx=False)["sqf"]
    assert (b <= a).all()


def test_int_and_float_arithmetic_agree_on_unit_sampling():
    rng = np.random.default_rng(23)
    mask = (rng.random((2, 2, 9, 8, 7)) < 0.9).astype(np.uint8)
    a = oracle.sep(mask, None, want_idx=False)
    # 1.0 + tiny is not "unit" for the oracle -> float64 path; values differ only at rounding level
    eps = 1.0 + 2.0**-40
    b = oracle.sep(mask, (eps, eps, eps), want_idx=False)
    assert b["sq"] is None
    np.testing.assert_allclose(b["sqf"], a["sq"].astype(np.float64), rtol=1e-10)
    assert np.array_equal(a["dist"], np.sqrt(a["sq"].astype(np.float64)))


def test_batch_independence():
    rng = np.random.default_rng(29)
    mask = (rng.random((3, 2, 6, 7)) < 0.8).astype(np.uint8)
    mask[1, 1] = 1  # one image with no background among normal ones
    full = oracle.sep(mask, (1.0, 2.0))
    for b in range(3):
        for c in range(2):
            one = oracle.sep(mask[b : b + 1, c : c + 1], (1.0, 2.0))
            assert np.array_equal(full["sqf"][b, c], one["sqf"][0, 0])
            assert np.array_equal(full["idx"][b, c], one["idx"][0, 0])
    assert np.isinf(full["dist"][1, 1]).all() and (full["idx"][1, 1] == -1).all()
    assert np.isfinite(full["dist"][0, 0]).all()


def test_values_greater_than_one_are_foreground():
    mask = np.array([[[0, 2, 255, 7, 0, 1]]], dtype=np.uint8)
    assert np.array_equal(oracle.sep(mask)["sq"][0, 0], [0, 1, 4, 1, 0, 1])


def test_no_background_per_image():
    mask = np.ones((1, 2, 3, 3), dtype=np.uint8)
    mask[0, 0, 1, 1] = 0
    r = oracle.sep(mask)
    assert np.isfinite(r["dist"][0, 0]).all()
    assert np.isinf(r["dist"][0, 1]).all()
    assert (r["sq"][0, 1] == np.iinfo(np.int64).max).all()
    assert (r["idx"][0, 1] == -1).all()


@pytest.mark.parametrize("shape,samp", [((40, 37), None), ((24, 20, 18), (2.5, 0.8, 1.0)), ((5, 6, 4, 7), None),
                                         ((3, 4, 3, 2, 3, 4), (1.0, 1.1, 1.2, 1.3, 1.4, 1.5))])
def test_scipy_black_box_values(shape, samp):
    """SciPy's distance_transform_edt, the paper's reference system (Results, 'Protocol'), agrees on
    values for images that contain background (its no-background convention differs and is not used)."""
    ndi = pytest.importorskip("scipy.ndimage")
    rng = np.random.default_rng(31 + len(shape))
    mask = (rng.random((2, 1) + shape) < 0.85).astype(np.uint8)
    r = oracle.sep(mask, samp, want_idx=False)
    for b in range(2):
        ref = ndi.distance_transform_edt(mask[b, 0], sampling=samp)
        np.testing.assert_allclose(r["dist"][b, 0], ref, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("shape,samp", [((7,), None), ((5, 6), None), ((4, 3, 5), (2.5, 0.8, 1.0)),
                                         ((3, 2, 4, 3), (1.0, 1.5, 0.5, 2.0)), ((2, 3, 2, 2, 3, 2, 2, 3), None)])
@pytest.mark.parametrize("kind", ["brute", "sep"])
def test_virtual_background_convention(shape, samp, kind):
    """Images without background under the virtual out-of-bounds convention (Section 2.3.2): pinned against the
    closed form d = sqrt((w_0 (x_0 + 1))^2 + sum_{k>=1} (w_k x_k)^2) with indices (-1, 0, .., 0), and against
    scipy.ndimage, whose convention it is.  Images with background in the same batch stay as they are."""
    ndi = pytest.importorskip("scipy.ndimage")
    ndim = len(shape)
    mask = np.ones((2, 1) + shape, dtype=np.uint8)
    mask[(1, 0) + tuple(n // 2 for n in shape)] = 0
    r = oracle.virtual_background(mask, samp, want_idx=True, kind=kind)
    w = np.ones(ndim) if samp is None else np.asarray(samp, dtype=np.float64)
    grid = np.meshgrid(*[np.arange(n) for n in shape], indexing="ij")
    sqf = (w[0] * (grid[0] + 1)) ** 2 + sum((w[k] * grid[k]) ** 2 for k in range(1, ndim))
    np.testing.assert_allclose(r["dist"][0, 0], np.sqrt(sqf), rtol=1e-13)
    if samp is None:
        assert np.array_equal(r["sq"][0, 0], (grid[0] + 1) ** 2 + sum(grid[k] ** 2 for k in range(1, ndim)))
    assert (r["idx"][0, 0][0] == -1).all() and (r["idx"][0, 0][1:] == 0).all()
    d_sp, i_sp = ndi.distance_transform_edt(mask[0, 0], sampling=samp, return_indices=True)
    np.testing.assert_allclose(r["dist"][0, 0], d_sp, rtol=1e-12)
    assert np.array_equal(r["idx"][0, 0], i_sp)
    plain = (oracle.brute if kind == "brute" else oracle.sep)(mask, samp)
    np.testing.assert_array_equal(r["dist"][1, 0], plain["dist"][1, 0])
    np.testing.assert_array_equal(r["idx"][1, 0], plain["idx"][1, 0])


# ---- far sites: the outward scan of the separable oracle walks tens to hundreds of rows before its cut-off ends it

@pytest.mark.parametrize("samp", [None, (2.5, 0.8, 1.0)], ids=["unit", "sampled"])
def test_far_single_site_closed_form(samp):
    """One background voxel in a 90 x 70 x 110 volume: every voxel's answer is the distance to that voxel, up to
    about 150 rows away, so a cut-off that stops a scan one row early (or a sign error far from the site) shows."""
    shape = (90, 70, 110)
    site = (71, 5, 93)
    mask = np.ones((1, 1) + shape, dtype=np.uint8)
    mask[(0, 0) + site] = 0
    r = oracle.sep(mask, samp)
    w = np.ones(3) if samp is None else np.asarray(samp, dtype=np.float64)
    grid = np.meshgrid(*[np.arange(n, dtype=np.float64) for n in shape], indexing="ij", sparse=True)
    sq = sum((w[k] * (grid[k] - site[k])) ** 2 for k in range(3))
    np.testing.assert_allclose(r["sqf"][0, 0], sq, rtol=1e-14, atol=0)
    np.testing.assert_allclose(r["dist"][0, 0], np.sqrt(sq), rtol=1e-14, atol=0)
    if samp is None:
        assert np.array_equal(r["sq"][0, 0], sq.astype(np.int64))
    for k in range(3):
        assert (r["idx"][0, 0, k] == site[k]).all()


def test_few_far_sites_against_brute_force_and_scipy():
    """Six background voxels in 60 x 50 x 70: scans of up to 70 rows whose winner changes along the way."""
    ndimage = pytest.importorskip("scipy.ndimage")
    rng = np.random.default_rng(424738)
    shape = (60, 50, 70)
    mask = np.ones((1, 1) + shape, dtype=np.uint8)
    for _ in range(6):
        mask[(0, 0) + tuple(int(rng.integers(0, n)) for n in shape)] = 0
    for samp in (None, (2.5, 0.8, 1.0)):
        s = oracle.sep(mask, samp)
        b = oracle.brute(mask, samp)
        np.testing.assert_allclose(s["sqf"], b["sqf"], rtol=1e-14, atol=0)
        ref = ndimage.distance_transform_edt(mask[0, 0], sampling=samp)
        np.testing.assert_allclose(s["dist"][0, 0], ref, rtol=1e-12, atol=1e-12)
        checker.check_indices(s["idx"], mask, b, samp)


def test_two_far_sites_long_lines_against_scipy():
    """Two background voxels in a 700 x 900 image: scans of several hundred rows on both axes."""
    ndimage = pytest.importorskip("scipy.ndimage")
    mask = np.ones((1, 1, 700, 900), dtype=np.uint8)
    mask[0, 0, 13, 880] = 0
    mask[0, 0, 650, 40] = 0
    for samp in (None, (0.7, 1.3)):
        s = oracle.sep(mask, samp)
        ref = ndimage.distance_transform_edt(mask[0, 0], sampling=samp)
        np.testing.assert_allclose(s["dist"][0, 0], ref, rtol=1e-12, atol=1e-12)
        w = np.ones(2) if samp is None else np.asarray(samp)
        yy, xx = np.meshgrid(np.arange(700.0), np.arange(900.0), indexing="ij")
        closed = np.minimum((w[0] * (yy - 13)) ** 2 + (w[1] * (xx - 880)) ** 2,
                            (w[0] * (yy - 650)) ** 2 + (w[1] * (xx - 40)) ** 2)
        np.testing.assert_allclose(s["sqf"][0, 0], closed, rtol=1e-14, atol=0)


def test_bad_arguments_are_rejected():
    with pytest.raises(RuntimeError):
        oracle.sep(np.ones((1, 1, 3), dtype=np.uint8), (0.0,))
    with pytest.raises(RuntimeError):
        oracle.sep(np.ones((1, 1, 3), dtype=np.uint8), (float("nan"),))
    with pytest.raises(RuntimeError):
        oracle.sep(np.ones((1, 1) + (2,) * 9, dtype=np.uint8))
    with pytest.raises(RuntimeError):
        oracle.sep_axes(np.ones((1, 1, 3, 3), dtype=np.uint8), [0, 0])


def test_empty_inputs():
    r = oracle.sep(np.ones((0, 1, 4), dtype=np.uint8))
    assert r["dist"].shape == (0, 1, 4)
    r = oracle.sep(np.ones((1, 1, 4, 0), dtype=np.uint8))
    assert r["dist"].size == 0
