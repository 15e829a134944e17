"""Parity of the fused erosion / dilation kernel (through the C ABI) against the numpy oracle: bit-exact, since
both sides do one float32 subtraction or addition per active position and exact minima / maxima."""
import zlib

import numpy as np
import pytest

from oracle import morph_oracle as mo
from paper_2608_24738_b200 import binding, buildlib

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    buildlib.build()
    binding.lib()


CASES = [
    ((2, 2, 37), (3,), None), ((1, 1, 37), (4,), (1,)), ((2, 1, 19, 23), (3, 3), None), ((1, 2, 19, 23), (2, 5), (0, -2)),
    ((1, 1, 40, 300), (7, 7), None), ((2, 1, 11, 12, 13), (3, 3, 3), None), ((1, 1, 11, 12, 13), (2, 3, 4), (0, -1, 1)),
    ((1, 1, 5, 6, 4, 7), (3, 2, 3, 3), (0, 0, 1, -1)), ((1, 1, 3, 4), (3, 3), None), ((1, 1, 2, 2, 2), (3, 3, 3), None),
    ((1, 1, 3, 3, 2, 3, 2, 3, 2, 3), (1, 3, 1, 2, 1, 3, 1, 2), None), ((1, 1, 6, 1, 9), (3, 1, 5), (1, 0, -2)),
    # last extent a multiple of 128: four voxels per lane in the interior kernel
    ((2, 1, 5, 128), (3, 3), None), ((1, 2, 3, 4, 256), (3, 3, 3), None), ((1, 1, 130, 384), (5, 4), (-1, 1)),
    ((3, 1, 128), (7,), (2,)), ((1, 1, 2, 3, 128), (3, 3, 5), (0, 0, -2)),
    # last extent a multiple of 32: binary masks run on bit-packed lines (one word per line, offsets up to +-31 along
    # the line, an element too wide for that, many images)
    ((2, 1, 9, 32), (3, 3), None), ((1, 1, 8, 64), (3, 41), None), ((1, 1, 4, 96), (2, 63), None), ((1, 1, 3, 64), (1, 65), None),
    ((5, 3, 6, 7, 64), (3, 2, 9), (0, 0, 3)),
    # the same with four lines per lane (extent before the last a multiple of 4), 1 to 4 axes, and 5 axes (byte kernels)
    ((2, 1, 12, 8, 64), (3, 3, 3), None), ((1, 1, 3, 4, 8, 32), (3, 2, 3, 5), (0, 0, 1, -1)), ((2, 2, 64), (5,), None),
    ((1, 1, 2, 3, 5, 32), (2, 3, 3, 3), None), ((1, 1, 2, 3, 4, 4, 32), (1, 3, 3, 2, 3), None), ((3, 1, 40, 160), (5, 5), (1, -1)),
    # rows of a multiple of 4 (from 32 voxels on): the last word of a line is ragged
    ((2, 1, 9, 36), (3, 3), None), ((1, 1, 8, 100), (3, 7), (0, 2)), ((1, 1, 5, 6, 44), (3, 3, 3), None), ((2, 1, 40, 1000), (5, 5), None),
    ((1, 2, 68), (9,), None),
]


def _element(fp_shape, seed, density=0.7):
    rng = np.random.default_rng(seed)
    fp = rng.random(fp_shape) < density
    fp.flat[rng.integers(0, fp.size)] = True
    return fp, rng.normal(size=fp_shape).astype(np.float32)


@pytest.mark.parametrize("shape,fp_shape,origin", CASES, ids=["x".join(map(str, c[0])) + "_" + "x".join(map(str, c[1])) for c in CASES])
@pytest.mark.parametrize("mode", mo.MODES)
def test_grey_erosion_and_dilation(shape, fp_shape, origin, mode):
    import torch

    seed = zlib.crc32(repr((shape, fp_shape, mode)).encode())
    img = np.random.default_rng(seed).normal(size=shape).astype(np.float32)
    fp, st = _element(fp_shape, seed + 1)
    t = torch.from_numpy(img).cuda()
    for structure in (None, st):
        for op, ref_fn in (("erosion", mo.grey_erosion), ("dilation", mo.grey_dilation)):
            got = binding.tm_grey_morph(t, fp, structure, op=op, mode=mode, cval=0.25, origin=origin)
            torch.cuda.synchronize()
            want = ref_fn(img, fp, structure, mode, 0.25, origin)
            assert np.array_equal(got.cpu().numpy(), want), (op, structure is not None)


@pytest.mark.parametrize("shape,fp_shape,origin", CASES, ids=["x".join(map(str, c[0])) + "_" + "x".join(map(str, c[1])) for c in CASES])
@pytest.mark.parametrize("border_value", [0, 1])
def test_binary_erosion_and_dilation(shape, fp_shape, origin, border_value):
    import torch

    seed = zlib.crc32(repr((shape, fp_shape, border_value)).encode())
    rng = np.random.default_rng(seed)
    fp, _ = _element(fp_shape, seed + 1)
    for density in (0.5, 0.95, 0.05):
        mask = (rng.random(shape) < density).astype(np.uint8) * rng.integers(1, 255, size=shape).astype(np.uint8)
        t = torch.from_numpy(mask).cuda()
        for op, ref_fn in (("erosion", mo.binary_erosion), ("dilation", mo.binary_dilation)):
            got = binding.tm_binary_morph(t, fp, op=op, border_value=border_value, origin=origin)
            torch.cuda.synchronize()
            assert np.array_equal(got.cpu().numpy(), ref_fn(mask, fp, border_value, origin)), op


def test_large_volume_against_the_oracle_and_scipy():
    """A volume of several tiles with a ragged tail (the benchmark's kind of input, smaller): 3^3 ball, all modes."""
    import torch

    ndi = pytest.importorskip("scipy.ndimage")
    img = np.random.default_rng(7).normal(size=(2, 1, 70, 81, 93)).astype(np.float32)
    fp = ndi.generate_binary_structure(3, 1)
    t = torch.from_numpy(img).cuda()
    for mode in mo.MODES:
        got = binding.tm_grey_morph(t, fp, None, op="erosion", mode=mode).cpu().numpy()
        assert np.array_equal(got, mo.grey_erosion(img, fp, None, mode))
        assert np.array_equal(got[1, 0], ndi.grey_erosion(img[1, 0], footprint=fp, mode=mode))
    b = torch.from_numpy((img > 0.5).astype(np.uint8)).cuda()
    got = binding.tm_binary_morph(b, fp, op="dilation").cpu().numpy()
    assert np.array_equal(got[0, 0].astype(bool), ndi.binary_dilation(img[0, 0] > 0.5, fp))


BOXES = [((2, 1, 19, 23), (5, 5), None), ((1, 2, 11, 12, 13), (3, 3, 3), None), ((1, 1, 20, 256), (4, 6), (-1, 2)),
         ((1, 1, 5, 6, 4, 7), (3, 2, 2, 2), (0, 0, -1, 0)), ((1, 1, 3, 4, 128), (3, 3, 3), (1, 0, -1)), ((1, 1, 4, 4), (5, 5), None)]


# contiguous extent a multiple of 4 and a window symmetric along it: the quad kernels for flat boxes (last two axes in
# one pass, one pass per earlier axis), with even sizes and origins on the other axes, rows of one quad, 1-D
# Flat boxes of odd extents, centred: the strip kernels (every border rule inside the kernel).  Shapes cover several
# strips and chunks, ragged last strips, axes shorter than the window, rows that are not a multiple of 128, unequal
# extents of the last two axes (two passes) and windows of one position on either axis; the last three (even extents
# or an origin) stay on the general kernels.
QUAD_BOXES = [((2, 1, 19, 24), (3, 3), None), ((1, 2, 11, 12, 16), (3, 3, 3), None), ((1, 1, 40, 64), (5, 9), None),
              ((1, 1, 7, 6, 5, 32), (3, 1, 3, 3), None), ((3, 1, 64), (5,), None), ((1, 1, 70, 132), (3, 3), None),
              ((1, 1, 67, 260), (5, 5), None), ((2, 1, 37, 140), (7, 7), None), ((1, 1, 35, 8), (9, 9), None),
              ((1, 1, 2, 4), (9, 9), None), ((1, 1, 3, 300), (7, 3), None), ((1, 1, 130, 12), (3, 1), None),
              ((1, 1, 21, 12), (1, 9), None), ((1, 1, 5, 3, 12), (7, 5, 3), None), ((1, 1, 66, 9, 8), (9, 1, 1), None),
              ((2, 1, 18, 17, 36), (5, 5, 5), None), ((1, 1, 1, 1, 4), (3, 3, 3), None), ((1, 2, 9, 21, 132), (3, 3, 3), None),
              ((1, 1, 13, 10, 260), (7, 7, 7), None), ((1, 1, 5, 9, 8), (9, 9, 9), None), ((2, 1, 3, 10, 11, 40), (3, 3, 3, 3), None),
              ((1, 1, 9, 10, 4), (4, 2, 1), (1, 0, 0)), ((1, 1, 6, 33, 8), (2, 6, 3), (0, -2, 0)), ((2, 1, 140, 260), (3, 7), (1, 0))]


@pytest.mark.parametrize("shape,fp_shape,origin", QUAD_BOXES, ids=["x".join(map(str, c[0])) + "_" + "x".join(map(str, c[1])) for c in QUAD_BOXES])
@pytest.mark.parametrize("mode", mo.MODES)
def test_full_box_elements_on_strip_kernels(shape, fp_shape, origin, mode):
    import torch

    seed = zlib.crc32(repr((shape, fp_shape, mode, "quadbox")).encode())
    img = np.random.default_rng(seed).normal(size=shape).astype(np.float32)
    fp = np.ones(fp_shape, dtype=bool)
    t = torch.from_numpy(img).cuda()
    for op, ref_fn in (("erosion", mo.grey_erosion), ("dilation", mo.grey_dilation)):
        got = binding.tm_grey_morph(t, fp, None, op=op, mode=mode, cval=0.25, origin=origin)
        assert np.array_equal(got.cpu().numpy(), ref_fn(img, fp, None, mode, 0.25, origin)), op
        if origin is None:
            passes = sum(1 for m in fp_shape[:-2] if m > 1)
            last2 = [m for m in fp_shape[-2:] if m > 1]
            passes += 2 if len(last2) == 2 and last2[0] != last2[1] else min(len(last2), 1)
            assert binding.tm_edt_last_launch_count() == passes


@pytest.mark.parametrize("seed", range(24))
def test_seeded_boxes_and_masks_on_the_strip_and_bit_kernels(seed):
    """Random shapes (rows a multiple of 4 for the strip kernels, of 32 for the bit-packed kernels), random odd boxes
    and border rules, against the oracle."""
    import torch

    rng = np.random.default_rng(777 + seed)
    ndim = int(rng.integers(1, 4))
    bits = bool(rng.integers(0, 2))
    last = (32 * int(rng.integers(1, 9)) if seed % 3 else 4 * int(rng.integers(8, 70))) if bits else 4 * int(rng.integers(1, 40))
    spatial = tuple(int(rng.integers(1, 40)) for _ in range(ndim - 1)) + (last,)
    shape = (int(rng.integers(1, 3)), int(rng.integers(1, 3))) + spatial
    fp_shape = tuple(int(rng.choice([1, 3, 5, 7, 9])) for _ in range(ndim))
    fp = np.ones(fp_shape, dtype=bool)
    mode = mo.MODES[int(rng.integers(0, len(mo.MODES)))]
    if bits:
        mask = (rng.random(shape) < float(rng.choice([0.3, 0.8, 0.97]))).astype(np.uint8)
        fp = rng.random(fp_shape) < 0.7
        fp.flat[int(rng.integers(0, fp.size))] = True
        b = torch.from_numpy(mask).cuda()
        for border_value in (0, 1):
            for op, ref_fn in (("erosion", mo.binary_erosion), ("dilation", mo.binary_dilation)):
                got = binding.tm_binary_morph(b, fp, op=op, border_value=border_value)
                assert np.array_equal(got.cpu().numpy(), ref_fn(mask, fp, border_value, None)), (shape, fp_shape, op)
    else:
        img = rng.normal(size=shape).astype(np.float32)
        t = torch.from_numpy(img).cuda()
        for op, ref_fn in (("erosion", mo.grey_erosion), ("dilation", mo.grey_dilation)):
            got = binding.tm_grey_morph(t, fp, None, op=op, mode=mode, cval=-1.5)
            assert np.array_equal(got.cpu().numpy(), ref_fn(img, fp, None, mode, -1.5, None)), (shape, fp_shape, mode, op)


@pytest.mark.parametrize("shape,fp_shape,origin", BOXES, ids=["x".join(map(str, c[0])) + "_" + "x".join(map(str, c[1])) for c in BOXES])
@pytest.mark.parametrize("mode", mo.MODES)
def test_full_box_elements_run_one_pass_per_axis(shape, fp_shape, origin, mode):
    """Flat full-box elements of 20 or more positions are decomposed into one line element per axis; the result
    must stay bit-identical to the oracle's single N-D minimum / maximum, for every border rule, origin and op."""
    import torch

    seed = zlib.crc32(repr((shape, fp_shape, mode, "box")).encode())
    rng = np.random.default_rng(seed)
    img = rng.normal(size=shape).astype(np.float32)
    fp = np.ones(fp_shape, dtype=bool)
    t = torch.from_numpy(img).cuda()
    for op, ref_fn in (("erosion", mo.grey_erosion), ("dilation", mo.grey_dilation)):
        got = binding.tm_grey_morph(t, fp, None, op=op, mode=mode, cval=-0.5, origin=origin)
        assert binding.tm_edt_last_launch_count() >= 1
        assert np.array_equal(got.cpu().numpy(), ref_fn(img, fp, None, mode, -0.5, origin)), op
    if mode == "constant":
        mask = (rng.random(shape) < 0.8).astype(np.uint8)
        b = torch.from_numpy(mask).cuda()
        for border_value in (0, 1):
            for op, ref_fn in (("erosion", mo.binary_erosion), ("dilation", mo.binary_dilation)):
                got = binding.tm_binary_morph(b, fp, op=op, border_value=border_value, origin=origin)
                assert np.array_equal(got.cpu().numpy(), ref_fn(mask, fp, border_value, origin)), (op, border_value)
