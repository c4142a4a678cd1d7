import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

GUARD_BYTES = 256
GUARD_VALUE = 0xA5


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


@pytest.fixture(scope="session")
def oracle_mod():
    import oracle

    oracle.set_threads(oracle.max_threads())
    return oracle


class GuardedAllocator:
    """Output allocator for the GPU tests: every output sits between two runs of GUARD_BYTES bytes that hold GUARD_VALUE,
    the second starting at the output's very last byte + 1; the output itself is pre-filled with the same value, so
    elements that a kernel fails to write differ from the oracle's.  `check()` asserts that no guard byte changed: the
    stand-in for a memory checker, which cannot be run on the shared GPUs."""

    def __init__(self):
        self.live = []

    def __call__(self, shape, dtype, device):
        import torch

        n = 1
        for d in shape:
            n *= int(d)
        nbytes = n * torch.empty((), dtype=dtype).element_size()
        raw = torch.full((GUARD_BYTES + nbytes + GUARD_BYTES,), GUARD_VALUE, dtype=torch.uint8, device=device)
        self.live.append((raw, nbytes, tuple(shape), dtype))
        return raw[GUARD_BYTES:GUARD_BYTES + nbytes].view(dtype).view(tuple(shape))

    def check(self):
        import torch

        torch.cuda.synchronize()
        live, self.live = self.live, []
        for raw, nbytes, shape, dtype in live:
            front, back = raw[:GUARD_BYTES], raw[GUARD_BYTES + nbytes:]
            assert bool((front == GUARD_VALUE).all()), "bytes before an output %s %s were overwritten" % (shape, dtype)
            assert bool((back == GUARD_VALUE).all()), "bytes after an output %s %s were overwritten" % (shape, dtype)
        return len(live)


@pytest.fixture(autouse=True)
def guard_outputs(request):
    """Every `gpu` test runs with guard bytes around every tensor the binding allocates (outputs, workspaces, expanded
    weights); they are checked when the test ends."""
    if request.node.get_closest_marker("gpu") is None:
        yield None
        return
    from paper_1908_05858_b200 import binding

    alloc = GuardedAllocator()
    prev = binding.set_output_allocator(alloc)
    try:
        yield alloc
        alloc.check()
    finally:
        binding.set_output_allocator(prev)
