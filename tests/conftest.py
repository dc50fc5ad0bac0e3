import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


@pytest.fixture(scope="session", autouse=True)
def _build_oracle():
    import oracle

    oracle.build()


@pytest.fixture
def knobs(monkeypatch):
    """Sets MQ_* environment knobs for one test.  The library reads each knob once, so it is told to read them again
    after every change and once more when the test's environment has been restored."""
    from paper_2609_28358_b200 import mq

    def set_knobs(**kv):
        for k, v in kv.items():
            monkeypatch.setenv(k, str(v))
        mq.reload_env()

    yield set_knobs
    monkeypatch.undo()
    mq.reload_env()
