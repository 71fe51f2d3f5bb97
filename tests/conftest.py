import os
import sys

import pytest

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")
    # the CUDA library is built in-tree and kept out of the history: (re)build it when it is
    # missing or older than its sources (a no-op otherwise); a missing library still fails loudly
    from paper_2406_03853_b200 import build as b
    try:
        b.build()
    except Exception:
        if not os.path.exists(b.LIB):
            raise


@pytest.fixture(scope="session")
def tiny_oracle():
    from tests.helpers import oracle_from_spec
    import eesd_synth as synth
    return oracle_from_spec(synth.TINY, max_ctx=160)
