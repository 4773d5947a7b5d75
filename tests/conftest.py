import sys
from pathlib import Path

import pytest

import os

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

# The library looks at its tuning / test switches (CONV2D_B200_*) only in a process started with this variable;
# several tests select kernel variants or inject faults through those switches.
os.environ.setdefault("CONV2D_B200_TUNING", "1")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


@pytest.fixture(scope="session")
def oracle():
    import oracle as _oracle
    _oracle.build()
    return _oracle
