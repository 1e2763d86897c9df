import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


def load_golden(name):
    """Parse a 'key: v v v' text fixture from tests/golden/ into {key: [ints]}."""
    out = {}
    for line in (ROOT / "tests" / "golden" / name).read_text().splitlines():
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, v = line.split(":")
        out[k.strip()] = [int(t) for t in v.split()]
    return out


@pytest.fixture(scope="session")
def golden():
    return load_golden
