import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


# ---- guard regions around every device buffer the binding allocates (GPU tests only) ------------------------
# Stand-in for a memory checker: each buffer handed to the library (cache, workspace, quantised buffer, outputs
# the binding creates) sits between two 64 KiB regions filled with a byte pattern; after every GPU test the
# regions of all buffers allocated during the test must still hold the pattern.  A kernel that writes a few
# bytes or a few rows past either end of a buffer fails the test that ran it.

GUARD_BYTES = 1 << 16
GUARD_PATTERN = 0xA5
GUARD_BUDGET = 60 << 30        # checked buffers are released early once this much is held


class GuardedAllocator:
    def __init__(self):
        self.live = []          # (outer tensor, payload bytes)
        self.held = 0
        self.violations = []

    def __call__(self, nbytes, device):
        import torch
        if self.held + nbytes > GUARD_BUDGET:
            self.check()
        outer = torch.empty(nbytes + 2 * GUARD_BYTES, dtype=torch.uint8, device=device)
        outer[:GUARD_BYTES].fill_(GUARD_PATTERN)
        outer[GUARD_BYTES + nbytes:].fill_(GUARD_PATTERN)
        self.live.append((outer, nbytes))
        self.held += nbytes
        return outer[GUARD_BYTES:GUARD_BYTES + nbytes]

    def check(self):
        """Verifies and releases every buffer allocated so far; returns the list of violations found so far."""
        import torch
        if self.live and torch.cuda.is_available():
            torch.cuda.synchronize()
        for outer, nbytes in self.live:
            lo = outer[:GUARD_BYTES]
            hi = outer[GUARD_BYTES + nbytes:]
            for name, g in (("before", lo), ("after", hi)):
                bad = (g != GUARD_PATTERN).nonzero()
                if bad.numel():
                    self.violations.append(f"{bad.numel()} guard byte(s) {name} a buffer of {nbytes} bytes changed "
                                           f"(first at offset {int(bad[0])} of the guard)")
        self.live.clear()
        self.held = 0
        return self.violations


@pytest.fixture(autouse=True)
def guard_device_buffers(request):
    if "gpu" not in request.keywords:
        yield
        return
    import torch
    if not torch.cuda.is_available():
        yield
        return
    from paper_2408_05646_b200 import build
    build.build_library()
    from paper_2408_05646_b200 import binding
    alloc = GuardedAllocator()
    saved = binding.device_alloc
    binding.device_alloc = alloc
    try:
        yield alloc
    finally:
        binding.device_alloc = saved
    violations = alloc.check()
    assert not violations, "; ".join(violations)


@pytest.fixture(autouse=True)
def report_distance_to_plain_oracle(request, record_property):
    """Tests whose oracle layer models the 16-bit cache (the storage hook) also measure the distance to the plain
    fp64 oracle (helpers.assert_close with an Expect); the largest such distance of a test goes into its report."""
    try:
        import helpers
    except Exception:
        yield
        return
    helpers.PLAIN_LOG.clear()
    yield
    if helpers.PLAIN_LOG:
        what, e_plain, e_kept = max(helpers.PLAIN_LOG, key=lambda t: t[1])
        record_property("max_abs_vs_plain_fp64_oracle", f"{e_plain:.3e} ({what}); with the storage hook {e_kept:.3e}")
        print(f"[plain oracle] {request.node.name}: max-abs {e_plain:.3e} at '{what}' (with the storage hook {e_kept:.3e})")
