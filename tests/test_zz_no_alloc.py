"""The entry point that allocates nothing (tm_edt_noalloc) against the ordinary one (tm_edt) and the CPU oracle.

Who needs it: callers that may not allocate device memory once they are running -- a loop with a memory
budget fixed at start-up, a process whose GPU memory belongs to another allocator.  Its scratch is a
fixed array inside the library that every call shares and that keeps the previous call's contents, so
the check is made on two calls in a row with different inputs: the second must not be disturbed by what
the first left behind.  This file sorts last so that a run stopping at the first failure has already run
every other test; it passes alone in a fresh process as well."""
import numpy as np
import pytest

import oracle
from paper_2608_24738_b200 import binding, buildlib, workloads
from tests import checker

pytestmark = pytest.mark.gpu


def _both(mask_np, sampling, dist, sq, idx):
    import torch

    t = torch.from_numpy(mask_np).cuda()
    a = binding.tm_edt_noalloc(t, sampling, return_distances=dist, return_sqdist=sq, return_indices=idx)
    b = binding.tm_edt(t, sampling, return_distances=dist, return_sqdist=sq, return_indices=idx)
    torch.cuda.synchronize()
    # and against the oracle, at the bars of the parity tests
    ref = oracle.sep(mask_np, sampling, want_idx=False)
    if dist:
        checker.check_dist(a["dist"].cpu().numpy(), ref["dist"])
    if sq:
        checker.check_sq_exact(a["sq"].cpu().numpy(), ref["sq"])
    if idx:
        checker.check_indices(a["idx"].cpu().numpy(), mask_np, ref, sampling)
    return a, b


def _same(a, b):
    # Same kernels on the same input: the distances agree far inside the parity tolerance
    # |d - d_ref| <= 1e-5 * max(1, d_ref); integer outputs agree exactly.
    if a["dist"] is not None:
        da, db = a["dist"].cpu().numpy().astype(np.float64), b["dist"].cpu().numpy().astype(np.float64)
        assert np.array_equal(np.isinf(da), np.isinf(db))
        fin = np.isfinite(db)
        assert (np.abs(da[fin] - db[fin]) <= 1e-5 * np.maximum(1.0, db[fin])).all()
    if a["sq"] is not None:
        assert np.array_equal(a["sq"].cpu().numpy(), b["sq"].cpu().numpy())
    if a["idx"] is not None:
        assert np.array_equal(a["idx"].cpu().numpy(), b["idx"].cpu().numpy())


def test_noalloc_matches_tm_edt_on_two_calls_in_a_row():
    buildlib.build()
    shape = (2, 1, 48, 64, 64)  # three passes: the built-in scratch is really used
    assert 0 < binding.tm_edt_workspace_bytes(shape) <= binding.tm_edt_noalloc_max_scratch()
    first = workloads.random_mask(101, shape, 0.9)
    second = workloads.random_mask(202, shape, 0.6)
    second[1] = 1  # an image without background in the second call
    a, b = _both(first, None, True, True, True)
    _same(a, b)
    a, b = _both(second, (2.5, 0.8, 1.0), True, False, True)
    _same(a, b)
    assert np.isinf(a["dist"][1].cpu().numpy()).all()
    # a four-axis problem (two scratch buffers) right after, then the first input again
    a, b = _both(workloads.random_mask(303, (1, 1, 6, 20, 24, 32), 0.8), None, True, True, True)
    _same(a, b)
    a, b = _both(first, None, True, True, True)
    _same(a, b)


def test_noalloc_refuses_what_does_not_fit():
    import torch

    buildlib.build()
    # three processed axes take 4 bytes of scratch per voxel: two volumes of 128^3 fill the 16 MiB array exactly,
    # a third one does not fit
    limit = binding.tm_edt_noalloc_max_scratch()
    fits, too_large = (2, 1, 128, 128, 128), (3, 1, 128, 128, 128)
    assert binding.tm_edt_workspace_bytes_for(fits) == 4 * 2 * 128 ** 3 == limit
    assert binding.tm_edt_workspace_bytes_for(too_large) > limit
    r = binding.tm_edt_noalloc(torch.zeros(fits, dtype=torch.uint8, device="cuda"))
    torch.cuda.synchronize()
    assert (r["dist"] == 0).all()
    t = torch.ones(too_large, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.TmEdtError) as ei:
        binding.tm_edt_noalloc(t)
    assert ei.value.status == binding.ERR_TOO_LARGE
    # problems without scratch (one or two fused axes) never touch the array and always fit
    r = binding.tm_edt_noalloc(torch.zeros((1, 1, 64, 64), dtype=torch.uint8, device="cuda"))
    torch.cuda.synchronize()
    assert (r["dist"] == 0).all()
