"""Sizes at the limits of the interface.

* A batch of more than 2^31 voxels: the library cuts it into image ranges of fewer than 2^31 voxels each, and every
  offset into the inputs and outputs is a 64-bit one.  The batch repeats a few distinct images, so the oracle transforms
  those once and every other image must equal its first copy bit for bit.
* One image of just under 2^31 voxels (the largest the interface accepts).  The oracle cannot transform it whole, so the
  result is checked through properties that hold at any size -- every index names a background voxel of the image at
  exactly the returned distance, background voxels name themselves, neighbouring distances differ by at most one voxel
  -- and, on windows cut out around sampled voxels, against the oracle itself: a window of half-width R around a voxel
  whose distance inside the window is at most R contains every candidate site, so the oracle's value there is the
  value of the whole image.
"""
import numpy as np
import pytest

import oracle
from paper_2608_24738_b200 import binding, workloads
from tests import checker

pytestmark = pytest.mark.gpu

REL_TOL = checker.REL_TOL


@pytest.fixture(autouse=True)
def _give_memory_back():
    """These cases hold tens of GiB: the caches of torch and of the library are emptied before and after each."""
    import gc
    import torch

    def release():
        gc.collect()
        torch.cuda.synchronize()
        torch.cuda.empty_cache()
        binding.tm_edt_trim_memory()

    release()
    yield
    release()


def _need_memory(gib):
    import torch

    free, _ = torch.cuda.mem_get_info()
    if free < gib * 2**30:
        pytest.skip("needs %d GiB of free device memory" % gib)


@pytest.mark.parametrize("kind", ["dist+sq", "sampling", "indices"])
def test_batch_of_more_than_2_31_voxels(kind):
    import torch

    _need_memory(100 if kind == "indices" else 40)
    spatial, distinct = (64, 128, 128), 4
    images = 2**31 // int(np.prod(spatial)) + 2 * distinct + 1  # 2057 images, 2.16e9 voxels, a ragged last range
    first = workloads.random_mask(77, (distinct, 1) + spatial, 0.97)
    first[2] = 1                      # an image without background
    first[3, 0, 10:50, 30:100, 5:120] = 1  # a block of foreground: distances up to 20
    sampling = (2.5, 0.8, 1.0) if kind == "sampling" else None
    ref = oracle.sep(first, sampling, want_idx=False)
    t = torch.from_numpy(first).cuda()[torch.arange(images, device="cuda") % distinct].contiguous()
    assert t.numel() > 2**31
    r = binding.tm_edt(t, sampling, return_distances=True, return_sqdist=kind == "dist+sq",
                       return_indices=kind == "indices")
    torch.cuda.synchronize()
    for name in ("dist", "sq", "idx"):
        out = r[name]
        if out is None:
            continue
        for k in range(distinct):
            copies = out[k::distinct]
            assert bool((copies == copies[:1]).all()), "image %d: a copy differs in %s" % (k, name)
    head = {name: (None if r[name] is None else r[name][:distinct].cpu().numpy()) for name in r}
    checker.check_dist(head["dist"], ref["dist"])
    if head["sq"] is not None:
        checker.check_sq_exact(head["sq"], ref["sq"])
    if head["idx"] is not None:
        checker.check_indices(head["idx"], first, ref, sampling)


def _coordinate(n, axis, ndim, start=0, device="cuda"):
    import torch

    shape = [1] * ndim
    shape[axis] = n
    return torch.arange(start, start + n, device=device, dtype=torch.int64).view(shape)


def _check_properties_on_device(mask_d, dist, sq, idx, spatial):
    """Slab by slab along the first axis; mask_d (n...), dist (n...), sq (n...) or None, idx (ndim, n...) or None."""
    import torch

    ndim, n0 = len(spatial), spatial[0]
    rows = max(1, (1 << 26) // (int(np.prod(spatial)) // n0))
    flat_mask = mask_d.reshape(-1)
    for a in range(0, n0, rows):
        b = min(n0, a + rows)
        m, d = mask_d[a:b], dist[a:b]
        bg = m == 0
        assert bool(torch.isfinite(d).all()) and bool((d[bg] == 0).all()) and bool((d[~bg] >= 1).all())
        s = None if sq is None else sq[a:b]
        if idx is not None:
            s_idx = torch.zeros(m.shape, dtype=torch.int64, device=m.device)
            flat = torch.zeros(m.shape, dtype=torch.int64, device=m.device)
            for k in range(ndim):
                ik = idx[k, a:b]
                assert int(ik.min()) >= 0 and int(ik.max()) < spatial[k]
                own = _coordinate(b - a if k == 0 else spatial[k], k, ndim, a if k == 0 else 0)
                s_idx += (own - ik) ** 2
                flat = flat * spatial[k] + ik
            assert bool((flat_mask[flat.reshape(-1)] == 0).all()), "an index names a foreground voxel"
            assert bool((s_idx[bg] == 0).all()), "a background voxel must name itself"
            if s is not None:
                assert torch.equal(s, s_idx)
            s = s_idx
        if s is not None:
            want = s.to(torch.float64).sqrt()
            assert bool(((d.to(torch.float64) - want).abs() <= REL_TOL * want.clamp(min=1.0)).all())
        # neighbouring voxels: distances differ by at most one voxel (with the slab's next row where there is one)
        e = dist[a:min(n0, b + 1)]
        for k in range(ndim):
            lo, hi = e.narrow(k, 0, e.shape[k] - 1), e.narrow(k, 1, e.shape[k] - 1)
            if lo.numel():
                assert float((hi - lo).abs().max()) <= 1.0 + 1e-4


def _check_windows_against_the_oracle(mask, dist_d, sq_d, spatial, points, radius):
    checked = 0
    for p in points:
        lo = [max(0, int(c) - radius) for c in p]
        hi = [min(n, int(c) + radius + 1) for c, n in zip(p, spatial)]
        crop = np.ascontiguousarray(mask[tuple(slice(l, h) for l, h in zip(lo, hi))])
        if crop.all():
            continue
        ref = oracle.sep(crop[None, None], None, want_idx=False)
        centre = tuple(int(c) - l for c, l in zip(p, lo))
        want_sq = int(ref["sq"][(0, 0) + centre])
        if want_sq > radius * radius:
            continue  # a nearer site may lie outside the window
        got = float(dist_d[tuple(int(c) for c in p)])
        assert abs(got - np.sqrt(want_sq)) <= REL_TOL * max(1.0, np.sqrt(want_sq)), (p, got, want_sq)
        if sq_d is not None:
            assert int(sq_d[tuple(int(c) for c in p)]) == want_sq, p
        checked += 1
    return checked


def _sample_points(rng, spatial, extra):
    pts = [tuple(0 for _ in spatial), tuple(n - 1 for n in spatial)]
    for corner in range(1, 2 ** len(spatial) - 1, 3):
        pts.append(tuple((n - 1) if (corner >> k) & 1 else 0 for k, n in enumerate(spatial)))
    pts += [tuple(int(rng.integers(0, n)) for n in spatial) for _ in range(400)]
    # the last rows of the image: the highest addresses
    pts += [tuple([spatial[0] - 1 - int(rng.integers(0, 2))] + [int(rng.integers(0, n)) for n in spatial[1:]]) for _ in range(100)]
    return pts + list(extra)


# spatial extents, index output (else squared distances), side of the foreground block, window half-widths
BIG = [((2047, 1024, 1024), True, 42, 8, 30), ((127, 128, 128, 1024), False, 20, 6, 13)]


@pytest.mark.parametrize("spatial,with_indices,side,near_radius,far_radius", BIG,
                         ids=["2047x1024x1024-indices", "127x128x128x1024-sq"])
def test_one_image_of_just_under_2_31_voxels(spatial, with_indices, side, near_radius, far_radius):
    import torch

    _need_memory(120)
    ndim = len(spatial)
    assert 2**31 - 2**25 <= int(np.prod(spatial)) < 2**31
    mask = workloads.large_random_mask(2024 + ndim, (1, 1) + spatial, 0.9)
    # a block of foreground at the far end of the image: scans of tens of rows across the highest addresses
    block = tuple(slice(n - 3 - side, n - 3) for n in spatial)
    mask[(0, 0) + block] = 1
    mask[(0, 0) + tuple(n - 1 for n in spatial)] = 1
    t = torch.from_numpy(mask).cuda()
    r = binding.tm_edt(t, None, return_distances=True, return_sqdist=not with_indices, return_indices=with_indices)
    torch.cuda.synchronize()
    dist = r["dist"][0, 0]
    sq = None if r["sq"] is None else r["sq"][0, 0]
    idx = None if r["idx"] is None else r["idx"][0, 0]
    _check_properties_on_device(t[0, 0], dist, sq, idx, spatial)
    rng = np.random.default_rng(5)
    centre = tuple(n - 3 - side // 2 for n in spatial)
    inside = [tuple(int(rng.integers(n - 3 - side, n - 3)) for n in spatial) for _ in range(40)]
    pts = _sample_points(rng, spatial, inside + [centre])
    near = _check_windows_against_the_oracle(mask[0, 0], dist, sq, spatial, pts[:-41], near_radius)
    far = _check_windows_against_the_oracle(mask[0, 0], dist, sq, spatial, pts[-41:], far_radius)
    assert near >= 450 and far >= 30
    assert float(dist[centre]) >= side // 2 - 1


def _repeated_batch(first, images):
    import torch

    distinct = first.shape[0]
    t = torch.from_numpy(first).cuda()[torch.arange(images, device="cuda") % distinct].contiguous()
    assert t.numel() > 2**31
    return t


def _every_copy_equals_the_first(out, want, distinct):
    """out: result of a batch that repeats `distinct` images; want: the oracle's result for those."""
    assert out.numel() > 2**31
    for k in range(distinct):
        copies = out[k::distinct]
        assert bool((copies == copies[:1]).all()), "image %d: a copy differs" % k
    assert np.array_equal(out[:distinct].cpu().numpy(), want)


@pytest.mark.parametrize("what", ["grey", "binary", "cdt"])
def test_morphology_and_cdt_on_batches_of_more_than_2_31_voxels(what):
    """tm_grey_morph, tm_binary_morph and tm_cdt take such a batch in one launch per pass (64-bit offsets)."""
    import torch
    from oracle import cdt_oracle as co
    from oracle import morph_oracle as mo

    _need_memory(40)
    spatial, distinct = ((256, 1024) if what == "cdt" else (512, 1024)), 3
    images = 2**31 // int(np.prod(spatial)) + 2 * distinct + 1
    rng = np.random.default_rng(99)
    box = np.ones((3, 3), dtype=bool)
    cross = np.array([[0, 1, 0], [1, 1, 1], [0, 1, 0]], dtype=bool)
    if what == "grey":
        first = rng.normal(size=(distinct, 1) + spatial).astype(np.float32)
        t = _repeated_batch(first, images)
        got = binding.tm_grey_morph(t, box, None, op="erosion", mode="reflect")
        _every_copy_equals_the_first(got, mo.grey_erosion(first, box, None, "reflect"), distinct)
        del got
        weights = rng.normal(size=(3, 3)).astype(np.float32)
        got = binding.tm_grey_morph(t, cross, weights, op="dilation", mode="nearest")
        _every_copy_equals_the_first(got, mo.grey_dilation(first, cross, weights, "nearest"), distinct)
    elif what == "binary":
        first = workloads.random_mask(31, (distinct, 1) + spatial, 0.8)
        t = _repeated_batch(first, images)
        got = binding.tm_binary_morph(t, box, op="erosion", border_value=1)
        _every_copy_equals_the_first(got, mo.binary_erosion(first, box, 1), distinct)
        del got
        got = binding.tm_binary_morph(t, cross, op="dilation", border_value=0)
        _every_copy_equals_the_first(got, mo.binary_dilation(first, cross, 0), distinct)
    else:
        first = workloads.random_mask(32, (distinct, 1) + spatial, 0.98)
        first[1] = 1  # an image without background
        first[2, 0, 100:160, 200:500] = 1
        t = _repeated_batch(first, images)
        for metric in ("chessboard", "taxicab"):
            got = binding.tm_cdt(t, metric)
            _every_copy_equals_the_first(got, co.separable(first, metric), distinct)
            del got
    torch.cuda.synchronize()
