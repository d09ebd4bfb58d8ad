import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


@pytest.fixture(scope="session", autouse=True)
def _library_built():
    """The shared library is built in-tree and is not under version control: (re)build it when it
    is missing or older than its sources (a no-op otherwise), so that a fresh checkout can run the
    tests.  Building is not a fallback: a failed build fails every test that needs the library."""
    from paper_2605_24058_b200 import build
    try:
        build.build_library()
    except Exception as e:          # no nvcc here: the tests that load the library will say so
        sys.stderr.write("liblordba.so was not (re)built: %s\n" % e)


@pytest.fixture(scope="session")
def oracle():
    import oracle as _oracle
    _oracle.build()
    return _oracle
