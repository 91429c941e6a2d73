import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def pytest_sessionstart(session):
    # the tests call the C ABI: make sure the in-tree libraries exist and are up to date (nvcc
    # cross-compiles without a GPU); a failure here is reported by the tests that load them
    try:
        from paper_2510_08522_b200 import build
        build.build(checked=True)
    except Exception as e:  # noqa: BLE001
        sys.stderr.write("conftest: building the CUDA libraries failed: %r\n" % (e,))
