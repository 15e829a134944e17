"""Parity of tm_cdt (bit-exact int32) and tm_bfdt (float32, relative 1e-5) against their oracles."""
import zlib

import numpy as np
import pytest

import oracle
from oracle import cdt_oracle as co
from paper_2608_24738_b200 import binding, buildlib, workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    buildlib.build()
    binding.lib()


SHAPES = [(2, 2, 1), (3, 1, 37), (2, 1, 19, 23), (1, 2, 40, 300), (1, 1, 1, 50, 1), (2, 1, 11, 12, 13), (1, 1, 5, 6, 4, 7),
          (1, 1, 3, 3, 2, 3, 2, 3, 2, 3), (1, 1, 260, 130), (1, 1, 6, 200, 33),
          (1, 1, 1100, 40), (1, 1, 3, 9000),  # beyond the shared-memory strip / the ballot-word row kernel
          # rows of a multiple of 32 voxels: the first two axes on 16-bit values (one to 32 words per row, segments of
          # the second axis that are empty, ragged and full, a third axis after them, an axis of one voxel in between)
          (2, 1, 64, 64), (3, 1, 5, 96), (1, 1, 300, 1024), (1, 2, 1024, 32), (2, 1, 7, 33, 64), (1, 1, 9, 1, 128),
          (1, 1, 70, 352), (2, 1, 1, 3, 160),
          # rows of a multiple of 4 from 64 voxels on: a ragged last word, 16-bit rows padded to whole words
          (2, 1, 100, 1000), (1, 1, 37, 500), (3, 1, 33, 68), (1, 1, 5, 6, 132), (2, 1, 70, 260), (1, 1, 3, 124)]


@pytest.mark.parametrize("shape", SHAPES, ids=["x".join(map(str, s)) for s in SHAPES])
@pytest.mark.parametrize("metric", ["taxicab", "chessboard"])
def test_cdt_matches_the_oracle(shape, metric):
    import torch

    for p_fg in (0.3, 0.9, 0.999):
        mask = workloads.random_mask(zlib.crc32(repr((shape, metric, p_fg)).encode()), shape, p_fg)
        if shape[0] > 1:
            mask[-1, -1] = 1  # an image without background
        if p_fg > 0.99:
            mask[0, 0].flat[7 % mask[0, 0].size] = 0
        got = binding.tm_cdt(torch.from_numpy(mask).cuda(), metric)
        torch.cuda.synchronize()
        assert got.dtype == torch.int32
        assert np.array_equal(got.cpu().numpy(), co.separable(mask, metric)), p_fg


def test_cdt_matches_scipy_on_a_larger_image():
    import torch

    ndi = pytest.importorskip("scipy.ndimage")
    w = workloads.config2()
    mask = w.mask[:2]
    t = torch.from_numpy(mask).cuda()
    for metric in ("taxicab", "chessboard"):
        got = binding.tm_cdt(t, metric).cpu().numpy()
        for b in range(2):
            assert np.array_equal(got[b, 0], ndi.distance_transform_cdt(mask[b, 0], metric=metric))


def test_cdt_at_the_benchmark_shape_against_scipy():
    """Two images of the benchmark's 1024^2 disk workload (32 pinned rows, 8 groups of 128 columns per image) and a
    volume whose third axis follows the two 16-bit passes."""
    import torch

    ndi = pytest.importorskip("scipy.ndimage")
    mask = workloads.config2(batch=2, size=1024, disks=80).mask
    vol = workloads.random_mask(77, (1, 1, 70, 100, 160), 0.97)
    for metric in ("taxicab", "chessboard"):
        got = binding.tm_cdt(torch.from_numpy(mask).cuda(), metric).cpu().numpy()
        for b in range(2):
            assert np.array_equal(got[b, 0], ndi.distance_transform_cdt(mask[b, 0], metric=metric))
        got = binding.tm_cdt(torch.from_numpy(vol).cuda(), metric).cpu().numpy()
        assert np.array_equal(got[0, 0], ndi.distance_transform_cdt(vol[0, 0], metric=metric))


@pytest.mark.parametrize("metric", ["taxicab", "chessboard"])
def test_cdt_structured_masks_on_the_sweep_path(metric):
    """Masks that stress the pinned rows / columns and the sweeps between them: one background voxel (scans and sweeps
    over the whole image), a background line, stripes of period 64 along either axis, a checkerboard of 48-voxel
    squares, and a batch whose second image has no background at all."""
    import torch

    shape = (2, 1, 200, 288)
    yy, xx = np.meshgrid(np.arange(shape[2]), np.arange(shape[3]), indexing="ij")
    cases = []
    one = np.ones(shape, dtype=np.uint8); one[0, 0, 199, 0] = 0; one[1, 0, 77, 131] = 0
    cases.append(one)
    line = np.ones(shape, dtype=np.uint8); line[0, 0, :, 130] = 0; line[1, 0, 63, :] = 0
    cases.append(line)
    stripes = np.ones(shape, dtype=np.uint8); stripes[0, 0][yy % 64 == 31] = 0; stripes[1, 0][xx % 64 == 0] = 0
    cases.append(stripes)
    board = np.ones(shape, dtype=np.uint8); board[:, 0] = (((yy // 48) + (xx // 48)) % 2).astype(np.uint8)
    cases.append(board)
    nobg = np.ones(shape, dtype=np.uint8); nobg[0, 0, 100, 100] = 0
    cases.append(nobg)
    for mask in cases:
        got = binding.tm_cdt(torch.from_numpy(mask).cuda(), metric).cpu().numpy()
        assert np.array_equal(got, co.separable(mask, metric))


@pytest.mark.parametrize("seed", range(24))
def test_cdt_seeded_shapes_around_the_piece_boundaries(seed):
    """Random shapes whose rows are a multiple of 32 voxels, with second extents around the 32-row pieces and row lengths
    around the 128-column groups of the sweep kernels, both metrics, against the oracle."""
    import torch

    rng = np.random.default_rng(4242 + seed)
    n0 = 32 * int(rng.integers(1, 11)) if seed % 2 == 0 else 4 * int(rng.integers(16, 90))
    n1 = int(rng.choice([1, 2, 31, 32, 33, 63, 64, 65, 95, 96, 97, int(rng.integers(3, 200))]))
    lead = [(), (int(rng.integers(2, 5)),)][int(rng.integers(0, 2))] if n0 * n1 < 20000 else ()
    shape = (int(rng.integers(1, 3)), int(rng.integers(1, 3))) + lead + (n1, n0)
    p_fg = float(rng.choice([0.5, 0.9, 0.99, 0.999]))
    mask = workloads.random_mask(int(rng.integers(0, 2**31)), shape, p_fg)
    if rng.random() < 0.3:
        mask[-1, -1] = 1  # an image without background
    t = torch.from_numpy(mask).cuda()
    for metric in ("taxicab", "chessboard"):
        got = binding.tm_cdt(t, metric).cpu().numpy()
        assert np.array_equal(got, co.separable(mask, metric)), (shape, p_fg, metric)


BF_SHAPES = [(2, 1, 40), (2, 2, 17, 23), (1, 1, 9, 10, 11), (1, 1, 4, 5, 3, 6), (1, 1, 30, 40)]


@pytest.mark.parametrize("shape", BF_SHAPES, ids=["x".join(map(str, s)) for s in BF_SHAPES])
@pytest.mark.parametrize("metric", ["euclidean", "taxicab", "chessboard"])
@pytest.mark.parametrize("sampled", [False, True])
def test_brute_force_transform(shape, metric, sampled):
    import torch

    ndim = len(shape) - 2
    sampling = tuple(0.5 + 0.75 * k for k in range(ndim)) if sampled else None
    mask = workloads.random_mask(zlib.crc32(repr((shape, metric)).encode()), shape, 0.9)
    if shape[0] > 1:
        mask[-1, -1] = 1
    got = binding.tm_bfdt(torch.from_numpy(mask).cuda(), sampling, metric).cpu().numpy()
    if metric == "euclidean":
        ref = oracle.brute(mask, sampling, want_idx=False)["dist"]
    else:
        ref = co.brute(mask, metric, sampling if sampled else (1.0,) * ndim)
    assert np.array_equal(np.isinf(got), np.isinf(ref))
    fin = np.isfinite(ref)
    assert (np.abs(got[fin] - ref[fin]) <= 1e-5 * np.maximum(1.0, ref[fin])).all()


def test_brute_force_validates_the_separable_transforms_on_the_device():
    """The use the paper names for the brute-force transform: the separable results, recomputed on the GPU."""
    import torch

    mask = torch.from_numpy(workloads.random_mask(5, (2, 1, 24, 40, 32), 0.95)).cuda()
    edt = binding.tm_edt(mask, (2.0, 1.0, 0.5))["dist"]
    assert torch.allclose(edt, binding.tm_bfdt(mask, (2.0, 1.0, 0.5), "euclidean"), rtol=1e-5, atol=1e-5)
    for metric in ("taxicab", "chessboard"):
        assert torch.equal(binding.tm_cdt(mask, metric).float(), binding.tm_bfdt(mask, None, metric))
