import gc
import os
import sys

import pytest

os.environ.setdefault("CUDA_MODULE_LOADING", "EAGER")   # see paper_2608_03839_b200/binding.py

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        have = torch.cuda.is_available()
    except Exception:
        have = False
    if have:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


# ---- guard zones (the stand-in for a memory checker) ------------------------------------
# Every GPU test runs with (1) each result tensor the binding allocates placed between two
# 256-byte margins of sentinel bytes, verified when the test ends, and (2) every pool created
# with sentinel bytes behind each of its device arrays, verified when the pool is closed or
# collected.  A kernel that writes one element past an output, a candidate list, the
# normalised queries or a staging block fails the test that ran it.
GUARD = 256
SENTINEL = 0x5A


class GuardedAllocator:
    def __init__(self):
        self.live = []          # (buffer, payload bytes)

    def __call__(self, shape, dtype, device):
        import torch
        if torch.device(device).type != "cuda":
            return torch.empty(shape, dtype=dtype, device=device)
        n = 1
        for s in shape:
            n *= int(s)
        nbytes = n * torch.empty((), dtype=dtype).element_size()
        buf = torch.full((GUARD + nbytes + GUARD,), SENTINEL, dtype=torch.uint8, device=device)
        self.live.append((buf, nbytes))
        return buf[GUARD:GUARD + nbytes].view(dtype).view(shape)

    def verify(self):
        import torch
        torch.cuda.synchronize()
        bad = []
        for buf, nbytes in self.live:
            lo, hi = buf[:GUARD], buf[GUARD + nbytes:]
            if not (bool((lo == SENTINEL).all()) and bool((hi == SENTINEL).all())):
                bad.append((nbytes, int((lo != SENTINEL).sum()), int((hi != SENTINEL).sum())))
        self.live.clear()
        return bad


@pytest.fixture(autouse=True)
def guard_zones(request):
    if "gpu" not in request.keywords:
        yield
        return
    from paper_2608_03839_b200 import binding as B
    alloc = GuardedAllocator()
    old_alloc, old_default = B.ALLOC, B.DEFAULT_DEBUG_GUARDS
    B.ALLOC, B.DEFAULT_DEBUG_GUARDS = alloc, True
    del B.GUARD_FAILURES[:]
    try:
        yield
        bad = alloc.verify()
        assert not bad, f"bytes outside an output tensor were written: {bad}"
        gc.collect()                      # pools the test dropped are checked as they go
        assert not B.GUARD_FAILURES, "a pool's guard zones were overwritten (see the traceback above)"
    finally:
        B.ALLOC, B.DEFAULT_DEBUG_GUARDS = old_alloc, old_default
        del B.GUARD_FAILURES[:]
