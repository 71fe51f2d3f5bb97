import os
import sys

import pytest

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")
    # the CUDA library is built in-tree and kept out of the history: (re)build it when it is
    # missing or older than its sources (a no-op otherwise).  A failed build is an error whenever a
    # build was needed: tests must never run against a library older than its sources.  Only a
    # machine without the compiler may go on with a library that is already up to date.
    from paper_2406_03853_b200 import build as b
    b.build()


@pytest.fixture(scope="session")
def tiny_oracle():
    from tests.helpers import oracle_from_spec
    import eesd_synth as synth
    return oracle_from_spec(synth.TINY, max_ctx=160)
