import os
import sys

import pytest

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


@pytest.fixture(scope="session")
def tiny_oracle():
    from tests.helpers import oracle_from_spec
    import eesd_synth as synth
    return oracle_from_spec(synth.TINY, max_ctx=160)
