"""The bounds-checked debug build (-DTM_EDT_DEBUG=1), this library's stand-in for a device memory checker: the quad
kernels check every shared-memory and global index, skip an access that leaves its range and report it through the
call's status.  Here the debug library runs shapes that take those kernels (three and four axes, aligned and ragged
tiles, images without background, far sites) and must report nothing while matching the oracle; a test hook that
hands the checks a bound that is too small shows that a violation does come back as a status, without any invalid
access ever being made."""
import numpy as np
import pytest

import oracle
from paper_2608_24738_b200 import binding, buildlib, workloads
from tests import checker

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _debug_library():
    buildlib.build(debug=True)
    binding.use_debug_library(True)
    try:
        assert binding.tm_edt_debug_build()
        yield
    finally:
        binding.use_debug_library(False)
        binding.lib()


SHAPES = [(2, 1, 33, 17, 40), (1, 2, 50, 128, 64), (1, 1, 128, 20, 48), (1, 1, 16, 40, 24, 32), (2, 1, 24, 40, 36),
          (1, 1, 100, 128, 128), (1, 1, 16, 64, 8, 8), (1, 1, 5, 6, 20, 28), (3, 1, 12, 16, 20), (1, 1, 7, 9, 4, 128)]


@pytest.mark.parametrize("shape", SHAPES, ids=["x".join(map(str, s)) for s in SHAPES])
def test_debug_build_reports_nothing_and_matches_the_oracle(shape):
    import torch

    ndim = len(shape) - 2
    for p_fg, sampling in ((0.8, None), (0.3, None), (0.97, (2.5, 0.8, 1.0, 1.25)[4 - ndim:]), (0.999, None)):
        mask = workloads.random_mask(sum(shape) + int(100 * p_fg), shape, p_fg)
        if shape[0] > 1:
            mask[-1] = 1  # an image without background
        unit = sampling is None
        ref = oracle.sep(mask, sampling, want_idx=False)
        t = torch.from_numpy(mask).cuda()
        for idx in (True, False):
            r = binding.tm_edt(t, sampling, return_distances=True, return_sqdist=unit, return_indices=idx)
            assert binding.tm_edt_debug_last_violation()[0] == 0
            checker.check_dist(r["dist"].cpu().numpy(), ref["dist"])
            if unit:
                checker.check_sq_exact(r["sq"].cpu().numpy(), ref["sq"])
            if idx:
                checker.check_indices(r["idx"].cpu().numpy(), mask, ref, sampling)


def test_a_violation_comes_back_as_a_status(switches):
    import torch

    t = torch.from_numpy(workloads.random_mask(5, (1, 1, 24, 40, 36), 0.8)).cuda()
    binding.tm_edt(t)
    switches.set("TM_EDT_DEBUG_INJECT", "1")
    with pytest.raises(binding.TmEdtError) as ei:
        binding.tm_edt(t)
    assert ei.value.status == binding.ERR_DEBUG_CHECK
    count, code, index, limit = binding.tm_edt_debug_last_violation()
    assert count > 0 and limit == 16 - 3 and index >= limit and code in (112, 121, 131)
    switches.set("TM_EDT_DEBUG_INJECT", None)
    r = binding.tm_edt(t)  # the context is intact and the next call is clean
    torch.cuda.synchronize()
    assert binding.tm_edt_debug_last_violation()[0] == 0 and torch.isfinite(r["dist"]).all()
