import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


def pytest_sessionstart(session):
    """Make sure the CUDA library is built in-tree (a no-op when it is up to date).  Without
    nvcc the library cannot be built; tests that need it then fail on import, loudly."""
    try:
        from paper_1901_03040_b200 import build
        build.build()
    except Exception as exc:  # noqa: BLE001
        print(f"conftest: could not build libqesgd.so: {exc}")
