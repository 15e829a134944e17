"""CPU oracle for the taxicab and chessboard distance transforms -- TEST INFRASTRUCTURE ONLY.

For every voxel of a (B, C, spatial...) mask, the distance to the nearest zero voxel of its image under
  taxicab     d1(x)   = min_s sum_k |x_k - s_k|
  chessboard  dinf(x) = min_s max_k |x_k - s_k|
(paper, Section 2.1; these are the metrics of its chamfer transform, Section 2.3.2, which reproduces
scipy.ndimage.distance_transform_cdt exactly).  Distances are int32; an image without background gets -1
everywhere, as SciPy returns.  `sampling` (brute force only) weighs the axes: sum_k w_k |.| and max_k w_k |.|, in
float64, +inf without background: the anisotropic case the paper reaches through its brute-force transform.

Two forms, both plain numpy:
  brute     the definition, every voxel against every background voxel (tiny inputs);
  separable nested per-axis exhaustive minima, g_k(x) = min_j op(g_{k-1}(x with x_k := j), |x_k - j|) with op = +
            for taxicab and max for chessboard; exact because both metrics combine the axes with an operation
            that distributes over the minimum.  No sweeps, no early exit.
Pins (tests/test_cdt_oracle_pins.py): each other, scipy.ndimage.distance_transform_cdt as a black box, closed
forms for a single background voxel, the ordering dinf <= d2 <= d1 <= ndim * dinf against the Euclidean oracle.
It shares no code with the CUDA library and never imports it.
"""
from __future__ import annotations

import numpy as np

BIG = np.int64(1) << 40


def _images(mask):
    mask = np.ascontiguousarray(mask)
    if mask.ndim < 3:
        raise ValueError("mask must be (B, C, spatial...)")
    return mask != 0


def brute(mask, metric, sampling=None):
    fg = _images(mask)
    spatial = fg.shape[2:]
    ndim = len(spatial)
    w = np.ones(ndim) if sampling is None else np.asarray(sampling, dtype=np.float64)
    grid = np.stack(np.meshgrid(*[np.arange(n) for n in spatial], indexing="ij"), axis=-1).reshape(-1, ndim)
    out = np.empty(fg.shape, dtype=np.float64 if sampling is not None else np.int32)
    for b in range(fg.shape[0]):
        for c in range(fg.shape[1]):
            sites = grid[~fg[b, c].reshape(-1)]
            if len(sites) == 0:
                out[b, c] = np.inf if sampling is not None else -1
                continue
            diff = np.abs(grid[:, None, :] - sites[None, :, :]) * w
            d = diff.sum(-1) if metric == "taxicab" else diff.max(-1)
            out[b, c] = d.min(1).reshape(spatial)
    return out


def separable(mask, metric):
    fg = _images(mask)
    ndim = fg.ndim - 2
    g = np.where(fg, BIG, np.int64(0))
    for k in range(ndim):
        ax = 2 + k
        n = g.shape[ax]
        pos = np.arange(n).reshape([n if a == ax else 1 for a in range(g.ndim)])
        best = np.full(g.shape, BIG, dtype=np.int64)
        for j in range(n):
            gj = np.take(g, [j], axis=ax)
            step = np.abs(pos - j)
            cand = gj + step if metric == "taxicab" else np.maximum(gj, step)
            best = np.minimum(best, cand)
        g = best
    out = np.where(g >= BIG, -1, g).astype(np.int32)
    return out
