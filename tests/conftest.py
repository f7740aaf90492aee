import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

GOLDEN = os.path.join(ROOT, "tests", "golden")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


def golden_rows(name):
    """Non-comment rows of a golden text fixture, split on whitespace."""
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if line:
                rows.append(line.split())
    return rows


@pytest.fixture(scope="session")
def oracle():
    import oracle as _oracle
    _oracle.build()
    return _oracle


class Guarded:
    """A device buffer with canary words on both sides, the stand-in for a memory checker: the
    kernels get the inner view; `check()` fails if anything outside it was written."""
    PAD = 64            # elements on each side (a multiple of 16 bytes for every dtype used)

    def __init__(self, torch, shape, dtype, fill=None):
        n = 1
        for d in shape:
            n *= int(d)
        self.torch = torch
        self.raw = torch.empty(n + 2 * self.PAD, dtype=dtype, device="cuda")
        self.bits = self.raw.view(torch.uint8)
        self.bits.fill_(0xA5)
        self.n, self.item = n, self.raw.element_size()
        self.view = self.raw[self.PAD:self.PAD + n].view(*shape)
        if fill is not None:
            self.view.fill_(fill)

    def check(self, what=""):
        lo = self.bits[: self.PAD * self.item]
        hi = self.bits[(self.PAD + self.n) * self.item:]
        assert bool((lo == 0xA5).all()) and bool((hi == 0xA5).all()), f"write outside {what or 'buffer'}"
