"""Seeded synthetic inputs for the distance-transform workloads.

This module holds input generators only -- no part of the transform's arithmetic -- so that the
CPU oracle and the CUDA path can both be fed from it without sharing any code of the method.
Every workload is produced on the host by ``numpy.random.default_rng(24738 + number)`` as a uint8
array of zeros (background) and ones (foreground) shaped (B, C, spatial...).

The paper's own benchmark inputs are described only by their sizes (Results, throughput table), so
these masks stand in for its "batched masks / volumes / volumetric time series": random pixels,
unions of disks, unions of ellipsoids, thresholded smooth noise, and a rank-8 stress case.
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass, field
from typing import Optional, Tuple

import numpy as np

SEED_BASE = 24738


@dataclass
class Workload:
    name: str
    number: int
    mask: np.ndarray  # (B, C, spatial...) uint8, C-contiguous
    sampling: Optional[Tuple[float, ...]]  # None = unit sampling
    want_dist: bool = True
    want_sq: bool = False
    want_idx: bool = False
    flat_index: bool = False  # index output as one linear index per voxel (a variant, not a benchmark default)
    note: str = ""
    meta: dict = field(default_factory=dict)

    @property
    def ndim(self) -> int:
        return self.mask.ndim - 2

    @property
    def voxels(self) -> int:
        return int(self.mask.size)

    def io_bytes(self) -> int:
        """Bytes the call must read and write: 1 per voxel in, 4 (f32) + 8 (i64) + 8*ndim out."""
        nidx = 1 if self.flat_index else self.ndim  # one linear index per voxel, or a coordinate per axis
        per = 1 + (4 if self.want_dist else 0) + (8 if self.want_sq else 0) + (8 * nidx if self.want_idx else 0)
        return per * self.voxels

    def sha256(self) -> str:
        return hashlib.sha256(self.mask.tobytes()).hexdigest()


def _guard_background(fg: np.ndarray) -> None:
    """Guarantee one background voxel per image: clear the first voxel if none is left."""
    if fg.all():
        fg[(0,) * fg.ndim] = False


def config1() -> Workload:
    """2-D single image 64x64, Bernoulli foreground p = 0.7, unit sampling, all three outputs."""
    rng = np.random.default_rng(SEED_BASE + 1)
    fg = rng.random((64, 64)) < 0.7
    return Workload("C1 2-D 64x64 Bernoulli(0.7)", 1, fg[None, None].astype(np.uint8), None, True, True, True)


def config2(batch: int = 32, size: int = 512, disks: int = 20) -> Workload:
    """2-D batch of 512x512 masks, each the union of 20 random disks (radius 10..60)."""
    rng = np.random.default_rng(SEED_BASE + 2)
    yy, xx = np.meshgrid(np.arange(size), np.arange(size), indexing="ij")
    out = np.zeros((batch, 1, size, size), dtype=np.uint8)
    for b in range(batch):
        centre = rng.uniform(0, size, (disks, 2))
        radius = rng.uniform(10, 60, disks)
        fg = np.zeros((size, size), dtype=bool)
        for (cy, cx), r in zip(centre, radius):
            fg |= (yy - cy) ** 2 + (xx - cx) ** 2 <= r * r
        _guard_background(fg)
        out[b, 0] = fg
    return Workload("C2 2-D %dx%dx%d disks" % (batch, size, size), 2, out, None)


def config3(batch: int = 8, channels: int = 2, size: int = 128, blobs: int = 8) -> Workload:
    """3-D volumes, union of 8 random axis-aligned ellipsoids (semi-axes 8..48), sampling (2.5, 0.8, 1.0)."""
    rng = np.random.default_rng(SEED_BASE + 3)
    zz, yy, xx = np.meshgrid(np.arange(size), np.arange(size), np.arange(size), indexing="ij", sparse=True)
    out = np.zeros((batch, channels, size, size, size), dtype=np.uint8)
    for b in range(batch):
        for c in range(channels):
            centre = rng.uniform(0, size, (blobs, 3))
            semi = rng.uniform(8, 48, (blobs, 3))
            fg = np.zeros((size, size, size), dtype=bool)
            for (cz, cy, cx), (az, ay, ax) in zip(centre, semi):
                fg |= ((zz - cz) / az) ** 2 + ((yy - cy) / ay) ** 2 + ((xx - cx) / ax) ** 2 <= 1.0
            _guard_background(fg)
            out[b, c] = fg
    return Workload("C3 3-D %dx%dx%d^3 ellipsoids" % (batch, channels, size), 3, out, (2.5, 0.8, 1.0))


def config4(batch: int = 2, frames: int = 16, size: int = 128) -> Workload:
    """4-D time series: N(0,1) noise smoothed with a Gaussian (sigma = 3 voxels on every axis),
    re-standardised to zero mean and unit variance per image, foreground where the field exceeds 0.3."""
    from scipy.ndimage import gaussian_filter  # input synthesis only

    rng = np.random.default_rng(SEED_BASE + 4)
    out = np.zeros((batch, 1, frames, size, size, size), dtype=np.uint8)
    for b in range(batch):
        z = rng.standard_normal((frames, size, size, size), dtype=np.float32)
        z = gaussian_filter(z, sigma=3.0)
        z = (z - z.mean()) / z.std()
        fg = z > 0.3
        _guard_background(fg)
        out[b, 0] = fg
    return Workload(
        "C4 4-D %dx%dx%d^3 smooth noise" % (batch, frames, size), 4, out, None, True, False, True
    )


def config5() -> Workload:
    """8-D stress: two images of 6^8 voxels; image 0 Bernoulli foreground p = 0.95, image 1 all foreground
    (no background at all: the +inf case).  Sampling 1.0, 1.1, .. 1.7 along the eight axes."""
    rng = np.random.default_rng(SEED_BASE + 5)
    shape = (6,) * 8
    out = np.ones((2, 1) + shape, dtype=np.uint8)
    out[0, 0] = rng.random(shape) < 0.95
    sampling = tuple((10 + k) / 10.0 for k in range(8))
    return Workload("C5 8-D 2x6^8 Bernoulli(0.95) + all-foreground", 5, out, sampling)


CONFIGS = {1: config1, 2: config2, 3: config3, 4: config4, 5: config5}


def random_mask(seed: int, shape, p_fg: float) -> np.ndarray:
    """Bernoulli(p_fg) foreground mask of the given (B, C, spatial...) shape, for the small parity cases."""
    rng = np.random.default_rng(seed)
    return (rng.random(tuple(shape)) < p_fg).astype(np.uint8)


def large_random_mask(seed: int, shape, p_fg: float) -> np.ndarray:
    """Bernoulli foreground mask for shapes of billions of voxels: one random byte per voxel, drawn in pieces,
    foreground where the byte is below round(256 p_fg)."""
    rng = np.random.default_rng(seed)
    out = np.empty(tuple(shape), dtype=np.uint8)
    flat = out.reshape(-1)
    threshold = int(round(256 * p_fg))
    piece = 1 << 26
    for start in range(0, flat.size, piece):
        n = min(piece, flat.size - start)
        flat[start:start + n] = rng.integers(0, 256, n, dtype=np.uint8) < threshold
    return out
