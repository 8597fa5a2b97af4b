import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HERE = os.path.dirname(os.path.abspath(__file__))
for p in (ROOT, HERE):
    if p not in sys.path:
        sys.path.insert(0, p)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a GPU box)")


@pytest.fixture(autouse=True)
def guarded_contexts_are_checked_when_closed(monkeypatch):
    """Every context a test creates guarded (tests/parity.py does so for all of its contexts) has its guard
    bands verified on the device when the test closes it: a kernel that wrote just outside one of the library's
    own buffers fails the test that made it do so."""
    from paper_1810_07354_b200 import api

    plain_close = api.ScarCheckpoint.close

    def close(self):
        if getattr(self, "ctx", None) and getattr(self, "guarded", False):
            bad = api.scar_ckpt_debug_check_guards(self.ctx)
            plain_close(self)
            assert bad == 0, f"{bad} guard bytes around the library's buffers were overwritten"
        else:
            plain_close(self)

    monkeypatch.setattr(api.ScarCheckpoint, "close", close)
    yield


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")
