"""Parity of the CUDA path (through the C ABI) against the CPU oracle, element by element.

Bars: int64 squared distances bit-exact; float32 distances |d - d_ref| <= 1e-5 * max(1, d_ref);
indices name a background voxel at the minimal distance (ties may differ from the oracle's pick)."""
import zlib

import numpy as np
import pytest

import oracle
from paper_2608_24738_b200 import binding, buildlib, workloads
from tests import checker

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    buildlib.build()
    binding.lib()


@pytest.fixture(params=["default", "generic", "no_lean"])
def path(request, switches):
    """Every kernel family: the planner's own choice, the rank-/extent-generic kernels forced, and the
    one-voxel-per-lane packed-entry kernels in place of the quad kernels."""
    switches.set("TM_EDT_FORCE_GENERIC", "1" if request.param == "generic" else None)
    switches.set("TM_EDT_NO_LEAN", "1" if request.param == "no_lean" else None)
    return request.param


def run_gpu(mask, sampling=None, dist=True, sq=False, idx=False, **kw):
    import torch

    t = torch.from_numpy(np.ascontiguousarray(mask)).cuda()
    r = binding.tm_edt(t, sampling, return_distances=dist, return_sqdist=sq, return_indices=idx, **kw)
    torch.cuda.synchronize()
    return {k: (None if v is None else v.cpu().numpy()) for k, v in r.items()}


def compare(mask, sampling, res, ref, dist=True, sq=False, idx=False):
    if dist:
        assert res["dist"].dtype == np.float32
        checker.check_dist(res["dist"], ref["dist"])
    if sq:
        checker.check_sq_exact(res["sq"], ref["sq"])
    if idx:
        checker.check_indices(res["idx"], mask, ref, sampling)


def full_check(mask, sampling=None):
    unit = sampling is None or all(float(s) == 1.0 for s in sampling)
    ref = oracle.sep(mask, sampling, want_idx=False)
    res = run_gpu(mask, sampling, dist=True, sq=unit, idx=True)
    compare(mask, sampling, res, ref, True, unit, True)
    return res, ref


SMALL = [
    (1, 1, 1), (1, 1, 5), (2, 3, 32), (1, 1, 33), (3, 1, 100), (1, 1, 129), (1, 1, 600), (1, 1, 1500),
    (1, 1, 7, 5), (2, 2, 33, 65), (1, 1, 1, 40), (1, 1, 40, 1), (1, 1, 130, 67), (1, 1, 67, 130), (1, 2, 64, 64),
    (1, 1, 9, 10, 11), (2, 1, 33, 17, 40), (1, 1, 5, 1, 6), (1, 1, 1, 1, 1), (1, 1, 140, 9, 12),
    (1, 1, 6, 5, 4, 7), (1, 1, 3, 4, 5, 3, 4), (1, 1, 2, 3, 4, 3, 2, 3), (1, 1, 3, 2, 3, 2, 3, 2, 3),
    (2, 1, 3, 2, 3, 2, 3, 2, 3, 4), (1, 1, 6, 6, 6, 6, 6, 6, 6, 6),
    (1, 1, 128, 128), (2, 1, 127, 128), (1, 1, 128, 100), (1, 2, 50, 128, 64), (1, 1, 128, 20, 48),
    (1, 1, 16, 40, 24, 32), (1, 1, 5, 6, 20, 7, 16), (1, 1, 3, 128, 1, 128),
    (2, 1, 3, 9, 5, 8), (1, 2, 20, 6, 7, 12), (2, 1, 2, 128, 4, 36),  # four axes on the quad kernels
    (2, 1, 200, 256), (1, 1, 129, 144), (1, 1, 300, 16), (1, 2, 512, 48), (1, 1, 1, 40, 1, 160),
    (1, 1, 1024, 48), (1, 1, 40, 1024), (2, 1, 600, 528), (1, 1, 513, 1008),
    (1, 1, 130, 48, 160), (1, 2, 20, 200, 64), (2, 1, 512, 6, 16), (1, 1, 9, 16, 512), (1, 1, 140, 1, 33, 1, 48),
]


def _sampling(ndim, kind):
    if kind == "unit":
        return None
    return tuple(0.5 + 0.37 * ((3 * k + 1) % 5) for k in range(ndim))


@pytest.mark.parametrize("shape", SMALL, ids=["x".join(map(str, s)) for s in SMALL])
@pytest.mark.parametrize("p_fg", [0.3, 0.9, 0.995])
@pytest.mark.parametrize("kind", ["unit", "sampled"])
def test_small_shapes_every_rank(shape, p_fg, kind, path):
    seed = zlib.crc32(repr((shape, p_fg, kind)).encode())
    mask = workloads.random_mask(seed, shape, p_fg)
    full_check(mask, _sampling(len(shape) - 2, kind))


TINY = [(37, 1, 5), (1, 1, 8), (70, 1, 3, 3), (3, 1, 8, 8, 8, 8), (2, 2, 7, 5, 3, 8, 2), (5, 1, 4, 4, 4, 4, 4),
        (1, 1, 2, 2, 2, 2, 2, 2, 2, 2), (1, 1, 8, 8, 8), (2, 1, 6, 1, 7, 1, 5, 6, 2), (1, 3, 5, 8, 7, 6, 5)]


@pytest.mark.parametrize("shape", TINY, ids=["x".join(map(str, s)) for s in TINY])
@pytest.mark.parametrize("kind", ["unit", "sampled"])
def test_extents_up_to_eight(shape, kind):
    """Every extent <= 8: axes are grouped (product of extents <= 256) and each group runs as one kernel over
    shared-memory tiles; the shapes split into groups at different places, leave ragged tiles along both the batch
    and the inner index, and cover line lengths 2..8.  Checked with the index map and, separately, distance only."""
    sampling = _sampling(len(shape) - 2, kind)
    for p_fg in (0.5, 0.97):
        mask = workloads.random_mask(zlib.crc32(repr((shape, kind, p_fg)).encode()), shape, p_fg)
        _, ref = full_check(mask, sampling)
        res = run_gpu(mask, sampling, dist=True, sq=False, idx=False)
        compare(mask, sampling, res, ref, True, False, False)
    mask = np.ones(shape, dtype=np.uint8)
    mask[-1].flat[-1] = 0  # one background voxel in the last image, none in the others
    full_check(mask, sampling)


FLAG_SHAPES = [(2, 1, 7), (2, 1, 300), (2, 1, 5, 6, 7, 130), (2, 1, 6, 5, 4, 7), (2, 1, 40, 36), (2, 1, 12, 20, 24), (2, 2, 6, 10, 12, 8),
               (2, 1, 140, 150), (2, 1, 1100, 40), (2, 1, 9, 9, 9, 9, 9, 9), (2, 1, 1, 30, 1, 20)]


@pytest.mark.parametrize("shape", FLAG_SHAPES, ids=["x".join(map(str, s)) for s in FLAG_SHAPES])
@pytest.mark.parametrize("kind", ["unit", "sampled"])
def test_flags_flat_index_and_virtual_background(shape, kind, path):
    """tm_edt_ex: one linear site index per voxel instead of coordinate planes, and the virtual-background
    values for images without background, on every kernel family.  Image 0 has background, image 1 has none."""
    sampling = _sampling(len(shape) - 2, kind)
    unit = sampling is None
    spatial = shape[2:]
    ndim = len(spatial)
    mask = workloads.random_mask(zlib.crc32(repr((shape, kind, "flags")).encode()), shape, 0.8)
    mask[1] = 1
    mask[0, 0].flat[3 % mask[0, 0].size] = 0
    ref = oracle.sep(mask, sampling, want_idx=False)
    stride0 = int(np.prod(spatial[1:]))

    def coords(flat):  # (C, n...) -> (C, ndim, n...)
        return np.stack(np.unravel_index(flat, spatial), axis=1)

    # flat index only
    res = run_gpu(mask, sampling, dist=True, sq=unit, idx=True, flat_index=True)
    assert res["idx"].shape == tuple(shape) and res["idx"].dtype == np.int64
    compare(mask, sampling, res, ref, True, unit, False)
    assert (res["idx"][1] == -1).all()
    checker.check_indices(coords(res["idx"][0])[None], mask[:1], {k: (None if v is None else v[:1]) for k, v in ref.items()},
                          sampling)
    # virtual background, coordinate planes
    vref = oracle.virtual_background(mask, sampling, want_idx=False)
    res = run_gpu(mask, sampling, dist=True, sq=unit, idx=True, virtual_background=True)
    checker.check_dist(res["dist"], vref["dist"])
    if unit:
        checker.check_sq_exact(res["sq"], vref["sq"])
    checker.check_indices(res["idx"][:1], mask[:1], {k: (None if v is None else v[:1]) for k, v in ref.items()}, sampling)
    assert (res["idx"][1][:, 0] == -1).all() and (res["idx"][1][:, 1:] == 0).all()
    # both flags, index output only
    res = run_gpu(mask, sampling, dist=False, sq=False, idx=True, virtual_background=True, flat_index=True)
    assert (res["idx"][1] == -stride0).all()
    checker.check_indices(coords(res["idx"][0])[None], mask[:1], {k: (None if v is None else v[:1]) for k, v in ref.items()},
                          sampling)


@pytest.mark.parametrize("shape", [(38, 1, 150, 256), (10, 1, 300, 1024), (2, 1, 140, 40, 160), (1, 2, 30, 520, 96),
                                   (5, 1, 1000, 1024)])  # the last: one block of 32 warps per SM (132 KB tile)
def test_16_bit_row_distances_feed_the_value_kernel(shape):
    """Batches large enough for the quad value kernel (at least 296 strips per axis), rows a multiple of 32, no index
    output: the first pass hands 16-bit row distances to it.  Rows without background, an image without background,
    dense and sparse masks; distances and exact squared distances."""
    for p_fg in (0.6, 0.995):
        mask = workloads.random_mask(zlib.crc32(repr((shape, p_fg, "d16")).encode()), shape, p_fg)
        mask[0, 0, 5:40] = 1   # rows without any background
        mask[-1, -1] = 1       # an image without background
        ref = oracle.sep(mask, None, want_idx=False)
        res = run_gpu(mask, None, dist=True, sq=True, idx=False)
        compare(mask, None, res, ref, True, True, False)
        assert binding.tm_edt_last_launch_count() == len(shape) - 2


@pytest.mark.parametrize("shape", [(1, 1, 64), (2, 1, 20, 30), (1, 2, 8, 9, 10), (1, 1, 200, 40)])
def test_degenerate_masks(shape, path):
    ndim = len(shape) - 2
    allfg = np.ones(shape, dtype=np.uint8)
    r = run_gpu(allfg, None, True, True, True)
    assert np.isinf(r["dist"]).all() and (r["dist"] > 0).all()
    assert (r["sq"] == np.iinfo(np.int64).max).all()
    assert (r["idx"] == -1).all()
    allbg = np.zeros(shape, dtype=np.uint8)
    r = run_gpu(allbg, None, True, True, True)
    assert (r["dist"] == 0).all() and (r["sq"] == 0).all()
    full_check(allbg, None)
    one = np.ones(shape, dtype=np.uint8)
    z = tuple(n // 3 for n in shape[2:])
    one[(0, 0) + z] = 0
    if shape[0] * shape[1] > 1:
        one[-1, -1] = 1  # last image keeps no background at all
        one[(-1, -1) + tuple(n - 1 for n in shape[2:])] = 0 if shape[0] * shape[1] > 2 else 1
    samp = tuple(1.0 + 0.25 * k for k in range(ndim))
    full_check(one, samp)
    full_check(one, None)
    # values above one are foreground too
    m = workloads.random_mask(5, shape, 0.7) * 200
    full_check(m.astype(np.uint8), None)


def test_mixed_batch_with_image_without_background(path):
    mask = workloads.random_mask(77, (3, 2, 20, 21, 22), 0.9)
    mask[1, 1] = 1
    res, ref = full_check(mask, (2.5, 0.8, 1.0))
    assert np.isinf(res["dist"][1, 1]).all()
    assert np.isfinite(res["dist"][0, 0]).all()


def test_half_space_and_far_sites(path):
    """Far sites are checked against the closed forms directly as well, not only against the oracle."""
    mask = np.ones((1, 1, 128, 96), dtype=np.uint8)
    mask[0, 0, :3] = 0
    rows = np.maximum(np.arange(128.0) - 2.0, 0.0)[:, None] * np.ones((1, 96))  # distance in rows to row 2
    res, _ = full_check(mask, None)
    assert np.array_equal(res["sq"][0, 0], (rows ** 2).astype(np.int64))
    res, _ = full_check(mask, (0.3, 1.9))
    np.testing.assert_allclose(res["dist"][0, 0], 0.3 * rows, rtol=1e-5, atol=1e-5)
    mask = np.ones((1, 1, 100, 128, 128), dtype=np.uint8)
    site = (99, 127, 0)
    mask[(0, 0) + site] = 0
    g = np.meshgrid(np.arange(100.0), np.arange(128.0), np.arange(128.0), indexing="ij", sparse=True)
    res, _ = full_check(mask, None)  # largest offsets an int8 carry can hold
    assert np.array_equal(res["sq"][0, 0], sum((g[k] - site[k]) ** 2 for k in range(3)).astype(np.int64))
    for k in range(3):
        assert (res["idx"][0, 0, k] == site[k]).all()
    res, _ = full_check(mask, (2.5, 0.8, 1.0))
    closed = np.sqrt(sum((w * (g[k] - site[k])) ** 2 for k, w in enumerate((2.5, 0.8, 1.0))))
    assert (np.abs(res["dist"][0, 0] - closed) <= 1e-5 * np.maximum(1.0, closed)).all()


@pytest.mark.parametrize("n", [512, 513, 1024, 1100, 2048])
def test_long_lines(n):
    """Extents above 128 use 16-bit offsets; unit sampling beyond 512 switches the envelope to float64."""
    mask = workloads.random_mask(n, (1, 1, 24, n), 0.97)
    mask[0, 0, :, : n // 2] |= workloads.random_mask(n + 1, (24, n // 2), 0.9995)
    full_check(mask, None)
    full_check(np.ascontiguousarray(mask.transpose(0, 1, 3, 2)), None)
    full_check(mask, (1.7, 0.6))


LONG = [(1, 1, 1100, 48), (2, 1, 48, 2064), (1, 1, 1040, 1056), (1, 1, 3000, 32), (1, 1, 16, 8192),
        (1, 1, 1100, 16, 32), (1, 2, 6, 1040, 48), (1, 1, 20, 32, 1040),
        (1, 1, 20, 32, 640), (1, 1, 600, 18, 50), (1, 1, 7, 800, 44), (2, 1, 500, 500), (1, 1, 1000, 999), (1, 1, 150, 150, 150),
        (1, 1, 6, 140, 20, 24), (1, 1, 130, 9, 10, 16), (2, 1, 4, 6, 8, 300), (1, 1, 5, 7, 520, 12)]


@pytest.mark.parametrize("shape", LONG, ids=["x".join(map(str, s)) for s in LONG])
@pytest.mark.parametrize("kind", ["unit", "sampled"])
def test_long_line_path(shape, kind):
    """Two or three axes with an extent above 128: shared-memory strips up to extent 1024 (integer keys while they
    fit 31 bits, float heights otherwise), cached height scans beyond, rows of any length and alignment in the
    first-axis pass.  Dense background and sparse background (long scans, rows without any background)."""
    sampling = _sampling(len(shape) - 2, kind)
    seed = zlib.crc32(repr((shape, kind)).encode())
    full_check(workloads.random_mask(seed, shape, 0.9), sampling)
    mask = np.ones(shape, dtype=np.uint8)
    rng = np.random.default_rng(seed)
    for _ in range(10):
        mask[(0, 0) + tuple(int(rng.integers(0, n)) for n in shape[2:])] = 0
    res, ref = full_check(mask, sampling)
    d = run_gpu(mask, sampling, dist=True, sq=False, idx=False)
    compare(mask, sampling, d, ref, True, False, False)


@pytest.mark.parametrize("pattern", ["left_edge", "top_edge", "disc", "frame", "diagonal"])
@pytest.mark.parametrize("kind", ["unit", "sampled"])
def test_long_line_far_sites(pattern, kind):
    """Long-line path with background far away (hundreds of rows): the block-wise far phase with its pruning by
    block minima, ties at the centre of a disc, sites on both sides."""
    n1, n0 = 1200, 1056
    yy, xx = np.mgrid[0:n1, 0:n0]
    mask = np.ones((n1, n0), dtype=np.uint8)
    if pattern == "left_edge":
        mask[:, 0] = 0
    elif pattern == "top_edge":
        mask[0, :] = 0
    elif pattern == "disc":
        mask = (((yy - n1 / 2) ** 2 + (xx - n0 / 2) ** 2) <= 500.0 ** 2).astype(np.uint8)
    elif pattern == "frame":
        mask[0, :] = 0; mask[-1, :] = 0; mask[:, 0] = 0; mask[:, -1] = 0
    else:
        mask[(yy * 7 + 3) % n1 == (xx * 5) % n1] = 0
        mask[300:900, :] = 1
    full_check(mask[None, None], _sampling(2, kind))


NARROW = [((1, 1, 1100, 2400), 2), ((1, 1, 2200, 1188), 2), ((1, 1, 4096, 1184), 2), ((1, 1, 1032, 2404), 2),
          ((2, 1, 1030, 40, 32), 3), ((1, 1, 1500, 40, 64), 3), ((1, 1, 4344, 1200), 2), ((1, 1, 4345, 600), 2),
          ((1, 1, 8192, 592), 2), ((1, 1, 2168, 2368), 2), ((1, 1, 2169, 1184), 2)]


@pytest.mark.parametrize("shape,launches", NARROW, ids=["x".join(map(str, s)) for s, _ in NARROW])
def test_long_axes_on_narrow_tiles(shape, launches):
    """Unit sampling without index output: an axis beyond 1024 rows runs on the quad value kernel with tiles of 16, 8
    or 4 columns (whole and ragged last tiles, two and three axes, the extents at which the tile width changes, the
    longest axis of the interface).  Dense background,
    blobs and a handful of sites (scans over thousands of rows), distances and exact squared distances."""
    import torch

    seed = zlib.crc32(repr(shape).encode())
    rng = np.random.default_rng(seed)
    dense = workloads.random_mask(seed, shape, 0.97)
    blobs = workloads.random_mask(seed + 1, shape, 0.999)
    sp = shape[2:]
    for _ in range(6):  # boxes of background
        lo = [int(rng.integers(0, n)) for n in sp]
        blobs[(slice(None), slice(None)) + tuple(slice(l, l + max(2, n // 5)) for l, n in zip(lo, sp))] = 0
    sparse = np.ones(shape, dtype=np.uint8)
    for _ in range(5):
        sparse[(0, 0) + tuple(int(rng.integers(0, n)) for n in sp)] = 0
    if shape[0] > 1:
        sparse[-1] = 1  # an image without background
    for mask in (dense, blobs, sparse):
        ref = oracle.sep(mask, None, want_idx=False)
        res = run_gpu(mask, None, dist=True, sq=True, idx=False)
        assert binding.tm_edt_last_launch_count() == launches
        compare(mask, None, res, ref, True, True, False)


FEW_COLUMNS = [(1, 1, 1024, 1024), (1, 1, 600, 800), (1, 1, 400, 2400), (1, 1, 384, 772), (1, 1, 500, 1000),
               (1, 1, 400, 24, 32), (1, 1, 2, 500, 800), (2, 1, 1000, 512)]


@pytest.mark.parametrize("shape", FEW_COLUMNS, ids=["x".join(map(str, s)) for s in FEW_COLUMNS])
def test_single_images_on_narrow_tiles(shape, switches):
    """A single image has too few columns to give every SM a 32-column tile of the value kernel: axes of 384 rows and
    more then run on tiles of 16 or 8 columns (16-bit row distances or 32-bit values in, final outputs or values out,
    ragged last tiles).  Distances and exact squared distances against the oracle, and squared distances bit-identical
    to the strip kernel such shapes ran on before."""
    seed = zlib.crc32(repr(shape).encode())
    rng = np.random.default_rng(seed)
    blobs = workloads.random_mask(seed, shape, 0.998)
    sp = shape[2:]
    for _ in range(5):
        lo = [int(rng.integers(0, n)) for n in sp]
        blobs[(slice(None), slice(None)) + tuple(slice(l, l + max(2, n // 4)) for l, n in zip(lo, sp))] = 0
    sparse = np.ones(shape, dtype=np.uint8)
    for _ in range(4):
        sparse[(0, 0) + tuple(int(rng.integers(0, n)) for n in sp)] = 0
    for mask in (workloads.random_mask(seed + 1, shape, 0.95), blobs, sparse):
        ref = oracle.sep(mask, None, want_idx=False)
        res = run_gpu(mask, None, dist=True, sq=True, idx=False)
        assert binding.tm_edt_last_launch_count() == len(sp)
        compare(mask, None, res, ref, True, True, False)
        switches.set("TM_EDT_NO_NARROW_TILES", "1")
        old = run_gpu(mask, None, dist=False, sq=True, idx=False)
        switches.set("TM_EDT_NO_NARROW_TILES", None)
        assert np.array_equal(old["sq"], res["sq"])


DECIMAL = [((4, 1, 512, 512), (0.8, 1.0), 2), ((2, 1, 300, 1024), (2.5, 1.0), 2), ((1, 1, 140, 40, 160), (2.5, 0.8, 1.0), 3),
           ((1, 1, 400, 24, 32), (1.25, 0.5, 2.0), 3), ((1, 1, 1024, 1024), (1.5, 0.5), 2), ((1, 1, 1100, 2400), (1.5, 0.5), 2),
           ((1, 1, 4096, 1184), (0.8, 1.0), 2), ((1, 1, 8192, 592), (1.0, 2.5), 2), ((1, 1, 1500, 40, 64), (2.0, 1.0, 0.5), 3),
           ((1, 1, 8192, 592), (1.0, 0.3), 3), ((2, 1, 200, 1000), (0.8, 1.0), 2),
           ((12, 1, 300, 1000), (0.8, 1.0), 2), ((12, 1, 300, 1008), (2.5, 1.0), 2), ((12, 1, 300, 496), (1.0, 0.5), 2)]


@pytest.mark.parametrize("shape,sampling,launches", DECIMAL,
                         ids=["x".join(map(str, s)) + "_" + "_".join(map(str, w)) for s, w, _ in DECIMAL])
def test_decimal_sampling_beyond_128_without_indices(shape, sampling, launches, switches):
    """Sampling whose squares share an integer scale, distances only, extents beyond 128: the value kernels run in exact
    scaled integers (16-bit row distances or integer heights first), on every tile width; a scale that would overflow 32
    bits, or too few tiles for the value kernel, stay on float heights; rows that are no multiple of 32 voxels get their
    weighted integer values from the other first-axis kernels (the last three cases).  Against the oracle, and against
    the float-height path."""
    seed = zlib.crc32(repr((shape, sampling)).encode())
    rng = np.random.default_rng(seed)
    blobs = workloads.random_mask(seed, shape, 0.998)
    sp = shape[2:]
    for _ in range(5):
        lo = [int(rng.integers(0, n)) for n in sp]
        blobs[(slice(None), slice(None)) + tuple(slice(l, l + max(2, n // 4)) for l, n in zip(lo, sp))] = 0
    sparse = np.ones(shape, dtype=np.uint8)
    for _ in range(4):
        sparse[(0, 0) + tuple(int(rng.integers(0, n)) for n in sp)] = 0
    if shape[0] > 1:
        sparse[-1] = 1  # an image without background
    for mask in (workloads.random_mask(seed + 1, shape, 0.9), blobs, sparse):
        ref = oracle.sep(mask, sampling, want_idx=False)
        res = run_gpu(mask, sampling, dist=True, sq=False, idx=False)
        assert binding.tm_edt_last_launch_count() == launches
        checker.check_dist(res["dist"], ref["dist"])
        switches.set("TM_EDT_NO_SCALED", "1")
        old = run_gpu(mask, sampling, dist=True, sq=False, idx=False)
        switches.set("TM_EDT_NO_SCALED", None)
        checker.check_dist(old["dist"], ref["dist"])


def test_sparse_background_long_axis_exactness():
    """Few background voxels and large extents: squared distances up to ~1e7 must stay exact."""
    mask = np.ones((1, 1, 2048, 300), dtype=np.uint8)
    rng = np.random.default_rng(3)
    for _ in range(12):
        mask[0, 0, rng.integers(0, 2048), rng.integers(0, 300)] = 0
    full_check(mask, None)


def test_sampling_without_a_common_integer_scale():
    """Sampling whose squares share no small integer scale stays on float32 heights; decimal sampling
    (handled in exact scaled integers) must agree with it within the distance tolerance."""
    import math

    mask = workloads.random_mask(31, (2, 1, 40, 64, 48), 0.9)
    full_check(mask, (math.pi / 3.0, math.sqrt(2.0), 1.0))
    full_check(mask, (2.5, 0.8, 1.0))
    mask4 = workloads.random_mask(32, (1, 1, 6, 24, 32, 16), 0.85)
    full_check(mask4, (math.e / 2.0, 1.0, math.sqrt(3.0), 0.9))
    full_check(mask4, (1.25, 1.0, 0.5, 2.0))


@pytest.mark.parametrize("shape", [(1, 1, 9, 4), (2, 1, 33, 8), (1, 1, 17, 12), (1, 2, 64, 20), (1, 1, 100, 124),
                                   (1, 1, 5, 128), (1, 1, 30, 16, 36), (1, 1, 300, 16), (1, 1, 77, 512)])
def test_any_nonzero_byte_is_foreground(shape):
    """Masks with arbitrary byte values (0x01, 0x7f, 0x80, 0xff ..): only 0 is background.  Exercises the
    zero-byte tests of the 4- and 16-voxels-per-lane first-axis passes."""
    rng = np.random.default_rng(zlib.crc32(repr(shape).encode()))
    vals = np.array([0, 1, 2, 0x7F, 0x80, 0x81, 0xFE, 0xFF], dtype=np.uint8)
    mask = vals[rng.integers(0, len(vals), size=shape)]
    mask[rng.random(shape) < 0.6] = 0xFF  # keep the background sparse
    full_check(mask, None)
    full_check(mask, tuple(1.0 + 0.5 * k for k in range(len(shape) - 2)))


def test_unaligned_input_pointer():
    """An input that does not start on a 4- or 16-byte boundary must take the byte-load kernels."""
    import torch

    for shape, samp in (((1, 1, 40, 64), None), ((1, 1, 12, 32, 64), (2.5, 0.8, 1.0)), ((1, 1, 200, 256), None)):
        mask = workloads.random_mask(41, shape, 0.85)
        ref = oracle.sep(mask, samp, want_idx=False)
        buf = torch.zeros(mask.size + 64, dtype=torch.uint8, device="cuda")
        for shift in (1, 3, 8):
            view = buf[shift: shift + mask.size].view(shape)
            view.copy_(torch.from_numpy(mask))
            assert view.data_ptr() % 16 != 0
            r = binding.tm_edt(view, samp, return_distances=True, return_indices=True)
            torch.cuda.synchronize()
            checker.check_dist(r["dist"].cpu().numpy(), ref["dist"])
            checker.check_indices(r["idx"].cpu().numpy(), mask, ref, samp)


def test_large_batches_run_as_image_ranges(switches):
    """A batch that does not fit one grid is cut into image ranges; a test hook makes the ranges tiny."""
    switches.set("TM_EDT_CHUNK_VOXELS", str(2 * 12 * 16 * 20 + 5))  # two images per range
    mask = workloads.random_mask(21, (5, 1, 12, 16, 20), 0.85)
    mask[3] = 1
    res, ref = full_check(mask, None)
    assert binding.tm_edt_last_launch_count() == 3 * 2  # three ranges, two kernels each
    full_check(mask, (1.5, 0.7, 1.0))
    switches.set("TM_EDT_FORCE_GENERIC", "1")
    full_check(mask, None)


def test_workspace_variant_and_preallocated_outputs():
    import torch

    mask = workloads.random_mask(9, (2, 2, 30, 31, 32), 0.8)
    ref = oracle.sep(mask, None, want_idx=False)
    t = torch.from_numpy(mask).cuda()
    ws = torch.empty(binding.tm_edt_workspace_bytes(mask.shape), dtype=torch.uint8, device="cuda")
    d = torch.full(mask.shape, -1.0, dtype=torch.float32, device="cuda")
    x = torch.full((2, 2, 3, 30, 31, 32), -7, dtype=torch.int64, device="cuda")
    r = binding.tm_edt(t, None, return_distances=True, return_indices=True, distances=d, indices=x, workspace=ws)
    torch.cuda.synchronize()
    assert r["dist"] is d and r["idx"] is x
    checker.check_dist(d.cpu().numpy(), ref["dist"])
    checker.check_indices(x.cpu().numpy(), mask, ref, None)
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.TmEdtError) as ei:
        binding.tm_edt(t, None, workspace=small)
    assert ei.value.status == binding.ERR_ALLOC


def test_pooled_scratch_and_trim():
    """tm_edt takes its scratch from the library's own memory pool; repeated calls reuse it and
    tm_edt_trim_memory hands it back without disturbing later calls."""
    import torch

    mask = workloads.random_mask(51, (2, 1, 40, 48, 64), 0.85)
    ref = oracle.sep(mask, None, want_idx=False)
    t = torch.from_numpy(mask).cuda()
    for _ in range(3):
        r = binding.tm_edt(t, None, return_distances=True, return_sqdist=True)
    torch.cuda.synchronize()
    checker.check_sq_exact(r["sq"].cpu().numpy(), ref["sq"])
    binding.tm_edt_trim_memory()
    r = binding.tm_edt(t, None, return_distances=True, return_sqdist=True)
    torch.cuda.synchronize()
    checker.check_sq_exact(r["sq"].cpu().numpy(), ref["sq"])
    binding.tm_edt_trim_memory()


def test_workspace_call_inside_a_cuda_graph():
    """tm_edt_ws only enqueues kernels (no allocation, no synchronisation), so it can be captured into a
    CUDA graph and replayed on new data in the same buffers."""
    import torch

    shape = (2, 1, 24, 40, 64)
    first = workloads.random_mask(61, shape, 0.85)
    second = workloads.random_mask(62, shape, 0.6)
    t = torch.from_numpy(first).cuda()
    ws = torch.empty(binding.tm_edt_workspace_bytes(shape), dtype=torch.uint8, device="cuda")
    d = torch.empty(shape, dtype=torch.float32, device="cuda")
    x = torch.empty(shape[:2] + (3,) + shape[2:], dtype=torch.int64, device="cuda")
    binding.tm_edt(t, None, distances=d, indices=x, workspace=ws)  # warm-up outside the capture
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        binding.tm_edt(t, None, distances=d, indices=x, workspace=ws, stream=torch.cuda.current_stream())
    for mask in (first, second):
        t.copy_(torch.from_numpy(mask))
        d.fill_(-1.0)
        g.replay()
        torch.cuda.synchronize()
        ref = oracle.sep(mask, None, want_idx=False)
        checker.check_dist(d.cpu().numpy(), ref["dist"])
        checker.check_indices(x.cpu().numpy(), mask, ref, None)


def test_side_stream_is_honoured():
    import torch

    mask = workloads.random_mask(10, (4, 1, 96, 96, 96), 0.8)
    ref = oracle.sep(mask, None, want_idx=False)
    t = torch.from_numpy(mask).cuda()
    s = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(s):
        r = binding.tm_edt(t, None, return_distances=True, return_sqdist=True)
        done = torch.cuda.Event()
        done.record(s)
    done.synchronize()
    checker.check_sq_exact(r["sq"].cpu().numpy(), ref["sq"])
    # explicit stream argument
    r = binding.tm_edt(t, None, return_distances=True, stream=s)
    s.synchronize()
    checker.check_dist(r["dist"].cpu().numpy(), ref["dist"])


def test_host_buffer_entry_point():
    import torch

    mask = workloads.random_mask(12, (2, 1, 40, 50), 0.85)
    ref = oracle.sep(mask, (1.5, 1.0), want_idx=False)
    t = torch.from_numpy(mask).pin_memory()
    r = binding.tm_edt_host(t, (1.5, 1.0), return_distances=True, return_indices=True)
    torch.cuda.synchronize()
    checker.check_dist(r["dist"].numpy(), ref["dist"])
    checker.check_indices(r["idx"].numpy(), mask, ref, (1.5, 1.0))
    with pytest.raises(binding.TmEdtError) as ei:
        binding.lib()  # keep the library loaded
        d = torch.empty(mask.shape, dtype=torch.float32, device="cuda")
        import ctypes

        shp = (ctypes.c_int64 * 4)(*mask.shape)
        rc = binding.lib().tm_edt_host(ctypes.c_void_p(t.data_ptr()), 2, shp, None, ctypes.c_void_p(d.data_ptr()),
                                       None, None, None)
        binding._check(rc)
    assert ei.value.status == binding.ERR_BAD_POINTER


def test_config1_brute_force_every_voxel(path):
    w = workloads.config1()
    ref = oracle.brute(w.mask, w.sampling)
    res = run_gpu(w.mask, None, True, True, True)
    compare(w.mask, None, res, ref, True, True, True)


@pytest.mark.parametrize("number", [2, 3, 4, 5])
def test_full_size_configs(number):
    w = workloads.CONFIGS[number]()
    ref = oracle.sep(w.mask, w.sampling, want_idx=False)
    res = run_gpu(w.mask, w.sampling, dist=w.want_dist, sq=w.want_sq, idx=w.want_idx)
    compare(w.mask, w.sampling, res, ref, w.want_dist, w.want_sq, w.want_idx)
    if number == 5:
        assert np.isinf(res["dist"][1]).all() and np.isfinite(res["dist"][0]).all()


def _fuzz_cases(count, seed):
    rng = np.random.default_rng(seed)
    extents = [1, 2, 3, 4, 5, 7, 8, 12, 16, 20, 31, 32, 33, 48, 64, 100, 128, 129, 200, 256]
    cases = []
    while len(cases) < count:
        ndim = int(rng.integers(1, 9))
        spatial = tuple(int(rng.choice(extents[: 9 if ndim > 4 else len(extents)])) for _ in range(ndim))
        bc = (int(rng.integers(1, 4)), int(rng.integers(1, 3)))
        if np.prod(spatial) * bc[0] * bc[1] > 250_000:
            continue
        kind = int(rng.integers(0, 3))
        if kind == 0:
            samp = None
        elif kind == 1:
            samp = tuple(float(rng.choice([0.5, 0.8, 1.0, 1.25, 2.0, 2.5])) for _ in range(ndim))
        else:
            samp = tuple(float(rng.uniform(0.3, 3.0)) for _ in range(ndim))
        p_fg = float(rng.choice([0.0, 0.3, 0.8, 0.97, 1.0]))
        cases.append((bc + spatial, samp, p_fg, int(rng.integers(0, 2**31))))
    return cases


@pytest.mark.parametrize("chunk", range(8))
def test_random_shapes_samplings_and_outputs(chunk):
    """Seeded differential fuzzing against the oracle: ranks 1..8, odd and aligned extents, batch and channel
    counts, unit / decimal / arbitrary sampling, empty and full masks, every output combination."""
    for shape, samp, p_fg, seed in _fuzz_cases(25, 1000 + chunk):
        mask = workloads.random_mask(seed, shape, p_fg)
        if p_fg not in (0.0, 1.0) and mask.shape[0] > 1:
            mask[-1, -1] = 1  # an image without background inside a normal batch
        try:
            full_check(mask, samp)
        except AssertionError as exc:  # name the case
            raise AssertionError("shape %r sampling %r p_fg %r seed %r: %s" % (shape, samp, p_fg, seed, exc))


def _large_extent_cases(count, seed):
    rng = np.random.default_rng(seed)
    big = [130, 131, 150, 257, 300, 500, 513, 1000, 1025, 1100, 2049]
    small = [1, 2, 3, 5, 8, 12, 16, 17, 33, 40]
    cases = []
    while len(cases) < count:
        ndim = int(rng.integers(2, 5))
        spatial = [int(rng.choice(small)) for _ in range(ndim)]
        for pos in rng.choice(ndim, size=int(rng.integers(1, 3)), replace=False):
            spatial[int(pos)] = int(rng.choice(big))
        bc = (int(rng.integers(1, 3)), 1)
        if np.prod(spatial) * bc[0] > 1_500_000:
            continue
        kind = int(rng.integers(0, 3))
        samp = None if kind == 0 else tuple(
            float(rng.choice([0.5, 0.8, 1.0, 2.5])) if kind == 1 else float(rng.uniform(0.4, 2.5)) for _ in range(ndim))
        p_fg = float(rng.choice([0.5, 0.9, 0.999]))
        cases.append((bc + tuple(spatial), samp, p_fg, int(rng.integers(0, 2**31))))
    return cases


@pytest.mark.parametrize("chunk", range(6))
def test_random_large_extents(chunk):
    """Seeded fuzzing of the paths beyond extent 128: two to four axes, one or two long axes with odd and aligned
    lengths in any position, dense to very sparse background."""
    for shape, samp, p_fg, seed in _large_extent_cases(8, 2000 + chunk):
        mask = workloads.random_mask(seed, shape, p_fg)
        if p_fg > 0.99:
            mask[0, 0].flat[seed % mask[0, 0].size] = 0  # at least one background voxel in the first image
        try:
            full_check(mask, samp)
        except AssertionError as exc:  # name the case
            raise AssertionError("shape %r sampling %r p_fg %r seed %r: %s" % (shape, samp, p_fg, seed, exc))


def _value_path_cases(count, seed):
    """Unit sampling without index output: shapes that take the value kernel on tiles of 32, 16, 8 or 4 columns."""
    rng = np.random.default_rng(seed)
    cases = []
    for _ in range(count):
        kind = int(rng.integers(0, 4))
        if kind == 0:    # one image, few columns, up to 1024 rows
            spatial = (int(rng.integers(384, 1025)), 4 * int(rng.integers(192, 600)))
        elif kind == 1:  # beyond 1024 rows
            n = int(rng.integers(1025, 8193))
            spatial = (n, 4 * int(rng.integers(148, max(149, min(700, 5_000_000 // (4 * n))))))
        elif kind == 2:  # three axes, the long one outermost or in the middle
            n = int(rng.integers(384, 3000))
            rest = (4 * int(rng.integers(2, 10)), 4 * int(rng.integers(8, 40)))
            spatial = (n,) + rest if rng.random() < 0.5 else (rest[0], n, rest[1])
        else:            # a batch of medium images
            spatial = (int(rng.integers(384, 700)), 32 * int(rng.integers(4, 17)))
        batch = int(rng.integers(2, 6)) if kind == 3 else 1
        cases.append(((batch, 1) + spatial, float(rng.choice([0.5, 0.9, 0.99, 0.9995])), int(rng.integers(0, 2**31))))
    return cases


@pytest.mark.parametrize("chunk", range(4))
def test_random_shapes_without_indices_beyond_128(chunk):
    """Seeded fuzzing of the value-carrying passes beyond extent 128 (the tile width follows the shape)."""
    for shape, p_fg, seed in _value_path_cases(6, 3000 + chunk):
        mask = workloads.random_mask(seed, shape, p_fg)
        mask[0, 0].flat[seed % mask[0, 0].size] = 0
        ref = oracle.sep(mask, None, want_idx=False)
        res = run_gpu(mask, None, dist=True, sq=True, idx=False)
        try:
            compare(mask, None, res, ref, True, True, False)
        except AssertionError as exc:  # name the case
            raise AssertionError("shape %r p_fg %r seed %r: %s" % (shape, p_fg, seed, exc))


F64_SHAPES = [(2, 1, 7), (2, 1, 40, 36), (2, 1, 12, 20, 24), (2, 1, 140, 150), (2, 1, 6, 5, 4, 7), (2, 1, 9, 9, 9, 9, 9, 9)]


@pytest.mark.parametrize("shape", F64_SHAPES, ids=["x".join(map(str, s)) for s in F64_SHAPES])
@pytest.mark.parametrize("kind", ["unit", "sampled"])
def test_float64_distances(shape, kind):
    """tm_edt_ex with float64 distances: recomputed in double precision from the chosen site, with the site taken
    from coordinate planes, from a flat index, or from scratch when no index output is requested.  Unit sampling:
    the correctly rounded root of the exact squared distance.  Image 1 has no background."""
    sampling = _sampling(len(shape) - 2, kind)
    unit = sampling is None
    mask = workloads.random_mask(zlib.crc32(repr((shape, kind, "f64")).encode()), shape, 0.85)
    mask[1] = 1
    mask[0, 0].flat[5 % mask[0, 0].size] = 0
    ref = oracle.sep(mask, sampling, want_idx=False)
    vref = oracle.virtual_background(mask, sampling, want_idx=False)

    def check(d, r):
        assert d.dtype == np.float64 and d.shape == tuple(shape)
        assert np.array_equal(np.isinf(d), np.isinf(r["dist"]))
        fin = np.isfinite(d)
        if unit:
            assert np.array_equal(d[fin], np.sqrt(r["sq"][fin].astype(np.float64)))
        else:
            np.testing.assert_allclose(d[fin], r["dist"][fin], rtol=2e-6, atol=0)

    for idx, flat in ((False, False), (True, False), (True, True)):
        res = run_gpu(mask, sampling, dist=True, sq=False, idx=idx, dist_f64=True, flat_index=flat)
        check(res["dist"], ref)
        res = run_gpu(mask, sampling, dist=True, sq=False, idx=idx, dist_f64=True, flat_index=flat, virtual_background=True)
        check(res["dist"], vref)


def test_strided_masks_are_gathered_by_the_library():
    """tm_edt_ex with byte strides: permuted, sliced and broadcast views give exactly what their contiguous copies
    give, and the oracle's values."""
    import torch

    base = torch.from_numpy(workloads.random_mask(77, (2, 3, 20, 24, 28), 0.9)).cuda()
    views = [
        base.permute(0, 1, 4, 2, 3),            # spatial axes permuted
        base[:, 1:3, ::2, :, 3:19],             # channel range, every second slice, a column range
        base[:, :1, 5:6].expand(2, 1, 7, 24, 28),  # a broadcast axis (stride 0)
        base.view(torch.bool)[:, :, :, ::3],    # bool mask, strided
    ]
    for v in views:
        assert not v.is_contiguous()
        got = binding.tm_edt(v, (1.5, 1.0, 0.5), return_indices=True, keep_strides=True)
        want = binding.tm_edt(v.contiguous(), (1.5, 1.0, 0.5), return_indices=True)
        torch.cuda.synchronize()
        assert torch.equal(got["dist"], want["dist"]) and torch.equal(got["idx"], want["idx"])
        m = v.contiguous().view(torch.uint8).cpu().numpy()
        ref = oracle.sep(m, (1.5, 1.0, 0.5), want_idx=False)
        checker.check_dist(got["dist"].cpu().numpy(), ref["dist"])
    # with a caller-provided workspace of the size the library reports
    v = views[0]
    nbytes = binding.tm_edt_ex_workspace_bytes(tuple(v.shape), tuple(v.stride()))
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    got = binding.tm_edt(v, None, return_sqdist=True, keep_strides=True, workspace=ws)
    want = binding.tm_edt(v.contiguous(), None, return_sqdist=True)
    torch.cuda.synchronize()
    assert torch.equal(got["sq"], want["sq"])


VALUE_SHAPES = [(2, 1, 12, 20, 24), (1, 2, 33, 17, 40), (1, 1, 128, 20, 48), (2, 1, 6, 10, 12, 8), (1, 1, 16, 40, 24, 32),
                (1, 1, 5, 6, 20, 7, 16), (1, 1, 3, 128, 1, 128), (1, 1, 128, 128, 128), (1, 1, 9, 10, 11),
                (3, 1, 40, 36), (1, 2, 128, 128), (2, 1, 7, 12), (2, 1, 1, 64, 1, 100)]  # two processed axes: the plane kernel is the last


@pytest.mark.parametrize("shape", VALUE_SHAPES, ids=["x".join(map(str, s)) for s in VALUE_SHAPES])
@pytest.mark.parametrize("kind", ["unit", "decimal", "two_decimals", "sampled"])
def test_outputs_without_indices(shape, kind, switches):
    """Without an index output the packed-entry path carries squared distances instead of offsets (16-bit values up to
    four axes, 32-bit beyond and in scaled-integer mode).  Distances and exact squared distances against the oracle,
    and bit-identical to what the offset-carrying kernels give."""
    ndim = len(shape) - 2
    # "two_decimals": squares with a common scale of 10000, beyond the 24 bits of the index-carrying keys but within
    # the 31 bits of plain values
    sampling = None if kind == "unit" else (tuple([2.5, 0.8, 1.0, 1.25, 0.5][:ndim]) if kind == "decimal" else
                                            (tuple([0.37, 0.8, 3.3, 1.25, 0.48][:ndim]) if kind == "two_decimals"
                                             else _sampling(ndim, "sampled")))
    unit = sampling is None
    for p_fg in (0.6, 0.98):
        mask = workloads.random_mask(zlib.crc32(repr((shape, kind, p_fg, "val")).encode()), shape, p_fg)
        if shape[0] > 1:
            mask[-1] = 1  # an image without background
        ref = oracle.sep(mask, sampling, want_idx=False)
        res = run_gpu(mask, sampling, dist=True, sq=unit, idx=False)
        compare(mask, sampling, res, ref, True, unit, False)
        if unit:
            only_sq = run_gpu(mask, sampling, dist=False, sq=True, idx=False)
            checker.check_sq_exact(only_sq["sq"], ref["sq"])
        switches.set("TM_EDT_NO_VALUE_CARRY", "1")
        old = run_gpu(mask, sampling, dist=True, sq=False, idx=False)
        switches.set("TM_EDT_NO_VALUE_CARRY", None)
        if kind in ("unit", "decimal"):  # integer paths: the same values either way
            assert np.array_equal(res["dist"], old["dist"])
        else:
            checker.check_dist(old["dist"], ref["dist"])
