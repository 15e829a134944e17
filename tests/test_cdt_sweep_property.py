"""The decomposition the chessboard / taxicab kernels of tm_cdt rely on, checked on the CPU against the oracle.

Second axis of the transform, given the row distances f (distance to the nearest background voxel inside the row):
  taxicab     g(y, x) = min_j f(j, x) + |y - j|
  chessboard  g(y, x) = min_j max(f(j, x), |y - j|)
The kernels compute g by two sweeps per piece of the image, a(y, x) = min(f(y, x), 1 + m(a(y - 1, .))) downwards and
the same upwards starting from a, with m = the value of the same column (taxicab) or the minimum over the three
neighbouring columns (chessboard), where the pieces are cut out by rows and columns whose exact values are computed
first ("pinned").  The claim: with exact values on the pinned voxels the sweeps are exact on every piece.  This file
emulates that scheme in numpy, with small pieces so that many paths cross pinned voxels, and compares with the oracle.
"""
import numpy as np
import pytest

from oracle import cdt_oracle as co

BIG = 1 << 20


def _row_distance(mask):
    """f: distance to the nearest zero inside the row (BIG for a row without any)."""
    h, w = mask.shape
    f = np.full((h, w), BIG, dtype=np.int64)
    for y in range(h):
        zeros = np.flatnonzero(mask[y] == 0)
        if zeros.size:
            f[y] = np.abs(np.arange(w)[:, None] - zeros[None, :]).min(axis=1)
    return f


def _sweeps_between_pins(f, exact, metric, seg, group):
    """Sweeps over pieces of (seg - 1) rows x group columns between pinned rows / columns taken from `exact`."""
    h, w = f.shape
    out = np.full((h, w), -7, dtype=np.int64)
    pinned_rows = sorted({min(h, (k + 1) * seg) - 1 for k in range((h + seg - 1) // seg)})
    chess = metric == "chessboard"

    def neighbours(prev, left, right):
        if not chess:
            return prev
        ext = np.concatenate(([left], prev, [right]))
        return np.minimum(np.minimum(ext[:-2], ext[1:-1]), ext[2:])

    for c0 in range(0, w, group):
        c1 = min(w, c0 + group)
        # pinned columns beside the piece (outside the image: nothing)
        lcol = exact[:, c0 - 1] if c0 > 0 else np.full(h, BIG)
        rcol = exact[:, c1] if c1 < w else np.full(h, BIG)
        top = -1
        for rp in pinned_rows:
            y0 = top + 1
            a = np.empty((rp - y0, c1 - c0), dtype=np.int64)
            prev = exact[y0 - 1, c0:c1] if y0 > 0 else np.full(c1 - c0, BIG)
            for i, y in enumerate(range(y0, rp)):  # down from the pinned row above
                le, ri = (lcol[y - 1], rcol[y - 1]) if y > 0 else (BIG, BIG)
                prev = np.minimum(f[y, c0:c1], 1 + neighbours(prev, le, ri))
                a[i] = prev
            prev = exact[rp, c0:c1]
            out[rp, c0:c1] = prev
            for i, y in reversed(list(enumerate(range(y0, rp)))):  # up from the own pinned row
                prev = np.minimum(a[i], 1 + neighbours(prev, lcol[y + 1], rcol[y + 1]))
                out[y, c0:c1] = prev
            top = rp
    return out


@pytest.mark.parametrize("metric", ["taxicab", "chessboard"])
@pytest.mark.parametrize("seg,group", [(2, 1), (3, 2), (4, 4), (8, 5), (32, 128)])
def test_sweeps_between_exact_pins_are_exact(metric, seg, group):
    rng = np.random.default_rng(1000 * seg + group + (7 if metric == "taxicab" else 0))
    for shape, p_fg in [((13, 17), 0.7), ((24, 9), 0.95), ((1, 12), 0.8), ((17, 1), 0.8), ((40, 33), 0.99), ((9, 20), 1.0)]:
        mask = (rng.random(shape) < p_fg).astype(np.uint8)
        if p_fg >= 1.0:
            mask[rng.integers(0, shape[0]), rng.integers(0, shape[1])] = 0  # one background voxel
        want = co.separable(mask[None, None], metric)[0, 0].astype(np.int64)
        f = _row_distance(mask)
        got = _sweeps_between_pins(f, want, metric, seg, group)
        assert np.array_equal(got, want), (shape, p_fg)


def test_column_recurrence_alone_is_not_exact_for_the_chessboard_metric():
    """Why the chessboard sweep needs the neighbouring columns: a running minimum along one column is wrong here."""
    mask = np.ones((6, 7), dtype=np.uint8)
    mask[0, 0] = 0
    want = co.separable(mask[None, None], "chessboard")[0, 0]
    f = _row_distance(mask)
    col = f[:, 3].copy()
    for y in range(1, 6):
        col[y] = min(col[y], col[y - 1] + 1)
    assert want[5, 3] == 5 and col[5] == 8
