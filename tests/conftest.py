import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the hand-written kernels through the C ABI)")


@pytest.fixture(autouse=True, scope="session")
def _plans_report_device_checks():
    """Every plan of the suite is asked for its device status words before it is destroyed.  A normal build
    records nothing (the call returns 0 without touching the device); a build with the index self-checks
    compiled in (`python -m paper_2609_29119_b200.build --debug-bounds`) fails the test that made an
    out-of-range access."""
    try:
        from paper_2609_29119_b200.binding import Plan
    except Exception:          # library not built: the tests that need it fail on their own
        yield
        return
    original = Plan.close

    def close_checked(self):
        if getattr(self, "handle", None) and getattr(self, "device", -1) >= 0:
            import torch
            torch.cuda.synchronize(self.device)
            status = self.check()
            original(self)
            assert status == 0, "the debug-bounds build recorded an out-of-range index (printed above)"
            return
        original(self)

    Plan.close = close_checked
    yield
    Plan.close = original
