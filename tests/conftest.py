import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch

        have_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        have_gpu = False
    if have_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


class _Switches:
    """Sets the library's debug switches (environment variables it reads once) and makes it read them again."""

    def __init__(self):
        self._saved = {}

    def set(self, name, value):
        from paper_2608_24738_b200 import binding

        self._saved.setdefault(name, os.environ.get(name))
        if value is None:
            os.environ.pop(name, None)
        else:
            os.environ[name] = str(value)
        binding.tm_edt_reload_switches()

    def restore(self):
        from paper_2608_24738_b200 import binding

        for name, old in self._saved.items():
            if old is None:
                os.environ.pop(name, None)
            else:
                os.environ[name] = old
        if self._saved:
            binding.tm_edt_reload_switches()
        self._saved = {}


@pytest.fixture
def switches():
    s = _Switches()
    yield s
    s.restore()


def read_golden(path):
    """Parse tests/golden/*.txt blocks into dicts (name, shape, sampling, mask, sq)."""
    import numpy as np

    cases, cur = [], {}
    with open(path) as fh:
        for raw in fh:
            line = raw.strip()
            if line.startswith("#"):
                continue
            if not line:
                if cur:
                    cases.append(cur)
                    cur = {}
                continue
            key, *vals = line.split()
            if key == "name":
                cur["name"] = vals[0]
            elif key == "shape":
                cur["shape"] = tuple(int(v) for v in vals)
            elif key == "sampling":
                cur["sampling"] = tuple(float(v) for v in vals)
            elif key == "mask":
                cur["mask"] = np.array([int(v) for v in vals], dtype=np.uint8)
            elif key == "sq":
                cur["sq"] = np.array([float(v) for v in vals], dtype=np.float64)
    if cur:
        cases.append(cur)
    for c in cases:
        c["mask"] = c["mask"].reshape((1, 1) + c["shape"])
        c["sq"] = c["sq"].reshape((1, 1) + c["shape"])
    return cases


GOLDEN_DIR = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
