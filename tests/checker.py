"""Comparison rules shared by the tests (no transform arithmetic beyond evaluating the definition
at a *given* candidate site, which is what the validity rule for indices needs)."""
import numpy as np

REL_TOL = 1e-5  # |d - d_ref| <= REL_TOL * max(1, d_ref) for float32 distances


def coords_grid(spatial):
    return np.meshgrid(*[np.arange(n, dtype=np.int64) for n in spatial], indexing="ij", sparse=True)


def check_dist(dist, ref_dist, tol=REL_TOL):
    dist = np.asarray(dist, dtype=np.float64)
    ref = np.asarray(ref_dist, dtype=np.float64)
    assert dist.shape == ref.shape
    inf_ref = np.isinf(ref)
    assert np.array_equal(np.isinf(dist), inf_ref), "infinite entries differ"
    assert not np.isnan(dist).any()
    fin = ~inf_ref
    err = np.abs(dist[fin] - ref[fin])
    bound = tol * np.maximum(1.0, ref[fin])
    bad = err > bound
    assert not bad.any(), "max excess %g at %d voxels" % ((err - bound).max(), int(bad.sum()))


def check_sq_exact(sq, ref_sq):
    sq = np.asarray(sq)
    assert sq.dtype == np.int64
    assert np.array_equal(sq, ref_sq), "%d squared distances differ" % int((sq != ref_sq).sum())


def check_indices(idx, mask, ref, sampling=None, tol=REL_TOL):
    """idx (B, C, ndim, n...) must name, for every voxel, a background voxel of the same image whose
    distance equals the reference minimum: exactly (integers) under unit sampling, within tol otherwise.
    Images without background must return -1 in every component."""
    mask = np.asarray(mask)
    idx = np.asarray(idx)
    B, C = mask.shape[:2]
    spatial = mask.shape[2:]
    ndim = len(spatial)
    assert idx.shape == (B, C, ndim) + spatial and idx.dtype == np.int64
    unit = sampling is None or all(float(s) == 1.0 for s in sampling)
    w = np.ones(ndim) if sampling is None else np.asarray(sampling, dtype=np.float64)
    grid = coords_grid(spatial)
    for b in range(B):
        for c in range(C):
            m = mask[b, c]
            ix = idx[b, c]
            if m.all():
                assert (ix == -1).all(), "image without background must give -1 indices"
                continue
            for k in range(ndim):
                assert ix[k].min() >= 0 and ix[k].max() < spatial[k], "index out of range"
            assert (m[tuple(ix[k] for k in range(ndim))] == 0).all(), "index names a foreground voxel"
            if unit:
                s = np.zeros(spatial, dtype=np.int64)
                for k in range(ndim):
                    s += (grid[k] - ix[k]) ** 2
                assert np.array_equal(s, ref["sq"][b, c]), "index is not at the minimal squared distance"
            else:
                s = np.zeros(spatial, dtype=np.float64)
                for k in range(ndim):
                    s += (w[k] * (grid[k] - ix[k])) ** 2
                d = np.sqrt(s)
                r = ref["dist"][b, c]
                assert (np.abs(d - r) <= tol * np.maximum(1.0, r)).all(), "index is not at the minimal distance"
            bgv = m == 0
            for k in range(ndim):
                own = np.broadcast_to(grid[k], spatial)
                assert np.array_equal(ix[k][bgv], own[bgv]), "background voxel must name itself"
