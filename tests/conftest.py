import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")
    # a fresh checkout has no built library yet (it is not tracked): build it once, in-tree
    try:
        from paper_2609_04609_b200 import build as libbuild

        libbuild.ensure_library()
    except Exception as e:  # the tests that need it will say so
        print(f"libciera.so could not be built: {e}", file=sys.stderr)


@pytest.fixture(scope="session")
def oracle():
    from oracle import ciera_oracle

    ciera_oracle.build()
    return ciera_oracle
