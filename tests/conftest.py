import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")
    # the library is built in-tree; rebuild only when a source is newer than the shared object
    from paper_2109_08751_b200 import build as lib_build

    lib_build.build()


@pytest.fixture(scope="session")
def golden_dir():
    return ROOT / "tests" / "golden"
