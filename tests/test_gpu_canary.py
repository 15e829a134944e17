"""Out-of-bounds writes, looked for without a memory checker: every output and the scratch of a call sit inside a
larger buffer filled with a canary byte, directly behind and in front of guard bytes; after the call the guards must
be untouched and the results must still match the oracle.  The scratch has exactly the size the library reports for
that call, so a kernel that writes past its own layout is caught as well.  Runs the shape lists of the parity tests on
every kernel family, with unit and other sampling, at 32-byte aligned and at merely element-aligned addresses."""
import numpy as np
import pytest

import oracle
from paper_2608_24738_b200 import binding, buildlib, workloads
from tests import checker
from tests.test_gpu_parity import LONG, SMALL, TINY

pytestmark = pytest.mark.gpu

CANARY = 0xA5
GUARD = 4096


@pytest.fixture(scope="module", autouse=True)
def _built():
    buildlib.build()
    binding.lib()


class Guarded:
    """`nbytes` of device memory between two guards of GUARD bytes; `skew` extra bytes shift the payload."""

    def __init__(self, nbytes, skew=0):
        import torch

        self.lo = GUARD + skew
        self.n = int(nbytes)
        self.buf = torch.full((self.lo + self.n + GUARD,), CANARY, dtype=torch.uint8, device="cuda")

    def view(self, dtype, shape):
        return self.buf[self.lo: self.lo + self.n].view(dtype).view(shape)

    def intact(self):
        return bool((self.buf[: self.lo] == CANARY).all()) and bool((self.buf[self.lo + self.n:] == CANARY).all())


def _run_guarded(mask, sampling, want_sq, skew):
    import torch

    shape = tuple(mask.shape)
    ndim = len(shape) - 2
    N = int(np.prod(shape))
    t = torch.from_numpy(mask).cuda()
    gd, gx = Guarded(4 * N, skew and 4), Guarded(8 * N * ndim, skew and 8)
    gs = Guarded(8 * N, skew and 8) if want_sq else None
    need = binding.tm_edt_workspace_bytes_for(shape, sampling, True, want_sq, True)
    gw = Guarded(max(need, 256))
    d = gd.view(torch.float32, shape)
    x = gx.view(torch.int64, shape[:2] + (ndim,) + shape[2:])
    s = gs.view(torch.int64, shape) if want_sq else None
    r = binding.tm_edt(t, sampling, return_distances=True, return_sqdist=want_sq, return_indices=True, distances=d,
                       sqdist=s, indices=x, workspace=gw.buf[gw.lo: gw.lo + gw.n])
    torch.cuda.synchronize()
    for name, g in (("distances", gd), ("indices", gx), ("squared distances", gs), ("scratch", gw)):
        assert g is None or g.intact(), "write outside the %s buffer" % name
    return {k: (None if v is None else v.cpu().numpy()) for k, v in r.items()}


SHAPES = SMALL + TINY + LONG + [(2, 1, 24, 40, 36), (1, 1, 16, 24, 8, 32), (1, 2, 128, 20, 32), (1, 1, 8, 16, 12, 64)]


@pytest.mark.parametrize("shape", SHAPES, ids=["x".join(map(str, s)) for s in SHAPES])
@pytest.mark.parametrize("family", ["default", "generic", "no_lean"])
def test_no_write_outside_outputs_and_scratch(shape, family, switches):
    switches.set("TM_EDT_FORCE_GENERIC", "1" if family == "generic" else None)
    switches.set("TM_EDT_NO_LEAN", "1" if family == "no_lean" else None)
    if family != "default" and int(np.prod(shape)) > 3_000_000:
        pytest.skip("large shapes on the planner's own choice only")
    mask = workloads.random_mask(sum(shape), shape, 0.8)
    ndim = len(shape) - 2
    for sampling in (None, tuple(0.5 + 0.37 * ((3 * k + 1) % 5) for k in range(ndim))):
        unit = sampling is None
        ref = oracle.sep(mask, sampling, want_idx=False)
        for skew in (0, 1):
            res = _run_guarded(mask, sampling, unit, skew)
            checker.check_dist(res["dist"], ref["dist"])
            if unit:
                checker.check_sq_exact(res["sq"], ref["sq"])
            checker.check_indices(res["idx"], mask, ref, sampling)


def test_distances_only_scratch_is_smaller_and_sufficient(switches):
    """Without an index output the wide-key and long-line paths carry no offsets: the per-call scratch is smaller
    and still never overrun."""
    import torch

    for shape in [(1, 1, 300, 320), (1, 1, 140, 150, 160), (1, 1, 1040, 1056), (1, 1, 6, 140, 20, 24)]:
        mask = workloads.random_mask(7, shape, 0.9)
        ref = oracle.sep(mask, None, want_idx=False)
        need = binding.tm_edt_workspace_bytes_for(shape, None, True, False, False)
        assert need < binding.tm_edt_workspace_bytes(shape)
        gw = Guarded(max(need, 256))
        N = int(np.prod(shape))
        gd = Guarded(4 * N)
        r = binding.tm_edt(torch.from_numpy(mask).cuda(), None, distances=gd.view(torch.float32, shape),
                           workspace=gw.buf[gw.lo: gw.lo + gw.n])
        torch.cuda.synchronize()
        assert gw.intact() and gd.intact()
        checker.check_dist(r["dist"].cpu().numpy(), ref["dist"])
