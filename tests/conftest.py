import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")
    # A fresh checkout has no built libraries (they are kept out of the history): build what is
    # missing or out of date.  nvcc cross-compiles without a GPU; the oracle needs only gcc.
    try:
        from paper_2510_03515_b200 import build as cuda_build
        cuda_build.build()
    except Exception as e:  # the tests that need the library will say so themselves
        print(f"[conftest] could not build librapid_pg.so: {e}", file=sys.stderr)


@pytest.fixture(scope="session")
def oracle():
    import oracle as _o
    _o.lib()
    return _o
